// Host-side tile-region planner (Section 4.2 of the paper): validation, map shapes, the
// equal partition of each group's output map, the receptive-field recursion of Eq. (1)
// generalised with explicit padding, sub-tiling for shared memory, workspace layout.
// Pure C++; no CUDA calls.
#include "plan.hpp"

#include <algorithm>
#include <cmath>
#include <cstring>

namespace ftp {

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int round4(int v) { return (v + 3) / 4 * 4; }
inline int extent(Span s) { return s.b - s.a + 1; }

// Inputs read by outputs o.a..o.b of a window op (kernel K, stride S, padding P), clamped to
// the input map.  For odd K, S = 1, P = K/2 this is Eq. (1) literally.
inline Span back_project(Span o, int K, int S, int P, int in_extent)
{
    Span s{o.a * S - P, o.b * S - P + K - 1};
    s.a = std::max(s.a, 0);
    s.b = std::min(s.b, in_extent - 1);
    return s;
}

inline int floor_div(int a, int b) { int q = a / b, r = a % b; return (r != 0 && ((r < 0) != (b < 0))) ? q - 1 : q; }
inline int ceil_div(int a, int b) { return -floor_div(-a, b); }

// Outputs that touch inputs i.a..i.b.  For odd K, P = K/2 this is Eq. (2) literally.
inline Span forward_project(Span i, int K, int S, int P, int out_extent)
{
    Span s{ceil_div(i.a + P - K + 1, S), floor_div(i.b + P, S)};
    s.a = std::max(s.a, 0);
    s.b = std::min(s.b, out_extent - 1);
    return s;
}

// Equal shares of a map's extent for the tiles (Section 4.2): part i of n owns [floor(i*E/n), floor((i+1)*E/n) - 1].
std::vector<Span> equal_partition(int a0, int len, int parts)
{
    std::vector<Span> out;
    for (int i = 0; i < parts; ++i) {
        long long lo = (long long)i * len / parts, hi = (long long)(i + 1) * len / parts - 1;
        out.push_back(Span{a0 + (int)lo, a0 + (int)hi});
    }
    return out;
}

struct AxisInfo {
    int n_ops;
    int K[kMaxOps], S[kMaxOps], P[kMaxOps];
    int ext[kMaxOps + 1];
};

void build_axis(AxisTables& t, const AxisInfo& ax, const std::vector<Span>& tiles, int split)
{
    const int n = ax.n_ops;
    std::vector<Span> cuts;
    t.tile_begin.clear();
    for (const Span& tl : tiles) {
        t.tile_begin.push_back((int)cuts.size());
        int len = extent(tl);
        int k = std::min(split, len);
        for (const Span& s : equal_partition(tl.a, len, k)) cuts.push_back(s);
    }
    t.tile_begin.push_back((int)cuts.size());
    t.count = (int)cuts.size();
    const int cnt = t.count;
    t.span.assign((size_t)(n + 1) * cnt * 2, 0);
    t.cell.assign((size_t)(n + 1) * cnt * 2, 0);
    t.maxext.assign(n + 1, 0);
    for (int r = 0; r < cnt; ++r) {
        Span s = cuts[r], c = cuts[r];
        for (int m = n; m >= 0; --m) {
            if (m < n) {
                s = back_project(s, ax.K[m], ax.S[m], ax.P[m], ax.ext[m]);
                c = Span{c.a * ax.S[m], c.b * ax.S[m] + ax.S[m] - 1};
            }
            t.span[((size_t)m * cnt + r) * 2 + 0] = s.a;
            t.span[((size_t)m * cnt + r) * 2 + 1] = s.b;
            t.cell[((size_t)m * cnt + r) * 2 + 0] = c.a;
            t.cell[((size_t)m * cnt + r) * 2 + 1] = c.b;
            t.maxext[m] = std::max(t.maxext[m], extent(s));
        }
    }
    t.scratch_off.assign(cnt + 1, 0);
    for (int r = 0; r < cnt; ++r)
        t.scratch_off[r + 1] = t.scratch_off[r] + (t.span[(size_t)r * 2 + 1] - t.span[(size_t)r * 2] + 1);
    t.cover.assign((size_t)ax.ext[0] * 2, 0);
    for (int pos = 0; pos < ax.ext[0]; ++pos) {
        int lo = -1, hi = -1;
        for (int r = 0; r < cnt; ++r)
            if (t.span[(size_t)r * 2] <= pos && pos <= t.span[(size_t)r * 2 + 1]) {
                if (lo < 0) lo = r;
                hi = r;
            }
        t.cover[(size_t)pos * 2] = lo;
        t.cover[(size_t)pos * 2 + 1] = hi;
    }
}

AxisInfo axis_info(const GroupPlan& g, bool y_axis)
{
    AxisInfo ax{};
    ax.n_ops = g.n_ops;
    for (int i = 0; i < g.n_ops; ++i) {
        const OpDesc& op = g.fwd_ops[i];
        ax.K[i] = op.keff; ax.S[i] = op.S; ax.P[i] = op.pad;
        ax.ext[i] = y_axis ? op.in_H : op.in_W;
        ax.ext[i + 1] = y_axis ? op.out_H : op.out_W;
    }
    return ax;
}

// Shared-memory geometry of the forward pass.  The input buffers of consecutive ops sit at
// opposite ends of the dynamic area (even ops at the bottom, odd ops at the top), so the area
// only has to hold the largest pair of neighbours.  Returns bytes incl. header.
size_t layout_forward(GroupPlan& g, const AxisTables& ty, const AxisTables& tx)
{
    int size[kMaxOps + 1] = {0};
    for (int i = 0; i < g.n_ops; ++i) {
        OpDesc& op = g.fwd_ops[i];
        int oh = ty.maxext[i + 1], ow = tx.maxext[i + 1];
        int bh = (oh - 1) * op.S + op.keff, bw = (ow - 1) * op.S + op.keff;
        op.in_pitch = bw;
        op.in_cs = bh * bw;
        size[i] = round4(op.cin * op.in_cs);
    }
    int total = 0;
    for (int i = 0; i < g.n_ops; ++i) total = std::max(total, size[i] + size[i + 1]);
    for (int i = 0; i < g.n_ops; ++i) g.fwd_ops[i].in_off = (i % 2 == 0) ? 0 : total - size[i];
    return (size_t)kSmemHeader + 4 * (size_t)total;
}

// Backward: while op i runs, the delta at its output (D_i), a copy of its input and the delta it
// produces (D_{i-1}) are alive.  Successive D buffers alternate between the two ends of the area
// and the input copy sits next to the bottom one, so the area holds the largest such triple.
// With dz_ch > 0 every fused conv+pool op also gets a staging area behind its input copy: the
// input-delta convolution then reads the delta at the conv output from there, dz_ch channels at a
// time, already routed through the arg-max and zero-extended by K - 1 on every side, instead of
// testing every value it reads (measured on B200: 29 % off the backward pass of such a group; for
// a plain conv, whose reads need one range test only, the staging costs more than it saves).
size_t layout_backward(GroupPlan& g, const AxisTables& ty, const AxisTables& tx, int dz_ch)
{
    const int n = g.n_ops;
    int dsize[kMaxOps], xsize[kMaxOps], zsize[kMaxOps];
    for (int i = 0; i < n; ++i) {
        OpDesc& op = g.bwd_ops[i];
        int oh = ty.maxext[i + 1], ow = tx.maxext[i + 1];
        int bh = (oh - 1) * op.S + op.keff, bw = (ow - 1) * op.S + op.keff;
        op.in_pitch = bw;
        op.in_cs = (bh * bw) | 1;       // odd channel stride: lanes that read consecutive channels hit distinct banks
        xsize[i] = round4(op.cin * op.in_cs);
        op.d_pitch = ow;
        op.d_cs = oh * ow;
        int dfl = round4(op.cout * op.d_cs);
        op.d_arg_off = dfl * 4;                       // relative to the D buffer, fixed up below
        dsize[i] = dfl + (op.kind == kOpConvPool ? round4((op.cout * op.d_cs + 3) / 4) : 0);
        // the input span is at most the input copy, and the staged delta K - 1 larger than the span
        op.dz_ch = op.kind == kOpConvPool ? std::min(dz_ch, op.cout) : 0;
        zsize[i] = round4(op.dz_ch * (bh + op.k - 1) * (bw + op.k - 1));
    }
    int total = 0;
    for (int i = 0; i < n; ++i) total = std::max(total, dsize[i] + xsize[i] + zsize[i] + (i > 0 ? dsize[i - 1] : 0));
    for (int i = 0; i < n; ++i) {
        OpDesc& op = g.bwd_ops[i];
        const bool low = ((n - 1 - i) % 2) == 0;
        op.d_off = low ? 0 : total - dsize[i];
        op.in_off = low ? dsize[i] : (i > 0 ? dsize[i - 1] : 0);
        op.dz_off = op.in_off + xsize[i];
        op.d_arg_off += op.d_off * 4;
    }
    return (size_t)kSmemHeader + 4 * (size_t)total;
}

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

// Tensor-core path.  A tile is [planes][Hp][Wp] entries of 16 bytes plus a tail of kTcTailEntries
// entries per plane.  The MMA operands address 16-row x 8-column pixel blocks (or runs of 16
// pixels) that may run past the rows and columns a tile really holds: such reads land in the
// following plane or tile and only reach accumulator rows that are discarded, so tiles carry no
// per-row padding; the activation area as a whole ends with a slack that keeps the furthest such
// read inside the block's shared memory.  Ping-pong placement as in layout_forward.  Bytes.
size_t tc_slack(int Wp, int planes_beyond, size_t plane_bytes)
{
    return ((size_t)16 * Wp + 32) * 16 + (size_t)planes_beyond * plane_bytes;
}

size_t layout_forward_tc(GroupPlan& g, const AxisTables& ty, const AxisTables& tx, int stages)
{
    size_t size[kMaxOps + 1] = {0}, slack = 0;
    for (int i = 0; i < g.n_ops; ++i) {
        OpDesc& op = g.fwd_ops[i];
        const int oh = ty.maxext[i + 1], ow = tx.maxext[i + 1];
        op.t_in_Hp = (oh - 1) * op.S + op.keff;
        op.t_in_Wp = (ow - 1) * op.S + op.keff;
        const size_t plane = tc_plane_bytes(op.t_in_Hp, op.t_in_Wp);
        size[i] = (size_t)(op.cin16 / 8) * plane;
        slack = std::max(slack, tc_slack(op.t_in_Wp, 0, plane));
    }
    size_t total = 0;
    for (int i = 0; i < g.n_ops; ++i) total = std::max(total, size[i] + size[i + 1]);
    for (int i = 0; i < g.n_ops; ++i) g.fwd_ops[i].t_in_off = (i % 2 == 0) ? 0 : (int)(total - size[i]);
    return (size_t)tc_fixed_bytes(stages) + total + slack;
}

// Tensor-core path, backward.  While op i runs, three tiles are alive: dz_i (delta at the conv output,
// before the pool, inside a zero apron of k-1), a copy of the op's input with the same pitch (the
// filter gradient contracts over runs of 16 pixels of both), and dz_{i-1} which the op produces.
// The filter-gradient operand spans 64 or 128 channels; channels beyond the real ones are reserved
// in the tile so that the operand stays inside it.
size_t layout_backward_tc(GroupPlan& g, const AxisTables& ty, const AxisTables& tx, int stages)
{
    const int n = g.n_ops;
    size_t dsize[kMaxOps], xsize[kMaxOps], slack = 0;
    for (int i = 0; i < n; ++i) {
        OpDesc& op = g.bwd_ops[i];
        const int oh = ty.maxext[i + 1], ow = tx.maxext[i + 1];
        if (op.kind == kOpPool) {
            op.t_dz_Hp = oh; op.t_dz_Wp = ow; op.t_dz_planes = op.cout16 / 8;
            op.t_x_Hp = 2 * oh; op.t_x_Wp = 2 * ow;
        } else {
            const int coh = op.S * oh, cow = op.S * ow, a = op.k - 1;
            op.t_dz_Hp = coh + 2 * a; op.t_dz_Wp = cow + 2 * a;
            op.t_dz_planes = op.cout16 <= 64 ? 8 : round_up(op.cout16, 128) / 8;
            op.t_x_Hp = coh + a; op.t_x_Wp = op.t_dz_Wp;
        }
        const size_t dplane = tc_plane_bytes(op.t_dz_Hp, op.t_dz_Wp);
        const size_t xplane = tc_plane_bytes(op.t_x_Hp, op.t_x_Wp);
        dsize[i] = (size_t)op.t_dz_planes * dplane;
        xsize[i] = (size_t)(op.cin16 / 8) * xplane;
        slack = std::max(slack, std::max(tc_slack(op.t_dz_Wp, 0, dplane), tc_slack(op.t_x_Wp, 0, xplane)));
    }
    size_t total = 0;
    for (int i = 0; i < n; ++i) total = std::max(total, dsize[i] + xsize[i] + (i > 0 ? dsize[i - 1] : 0));
    for (int i = 0; i < n; ++i) {
        OpDesc& op = g.bwd_ops[i];
        const bool low = ((n - 1 - i) % 2) == 0;
        op.t_dz_off = low ? 0 : (int)(total - dsize[i]);
        op.t_x_off = low ? (int)dsize[i] : (int)(i > 0 ? dsize[i - 1] : 0);
    }
    return (size_t)tc_fixed_bytes(stages) + total + slack;
}

void count_macs(const GroupPlan& g, const PassPlan& pp, double* done, double* untiled);

// Sub-tiling of one pass: the smallest split (largest sub-tile) whose buffers fit the shared-memory
// budget; for the forward pass, whose sub-tile stacks are spread over all SMs, a slightly finer
// split is taken instead when it fills the last round of blocks better (estimated time = rounds of
// blocks x multiply-accumulates of one stack, halo recomputation included).
int choose_subtiles(GroupPlan& g, bool backward, const PlanOpts& o, int N)
{
    const AxisInfo ay = axis_info(g, true), ax = axis_info(g, false);
    int max_h = 0, max_w = 0;
    for (const Span& s : g.tile_y) max_h = std::max(max_h, extent(s));
    for (const Span& s : g.tile_x) max_w = std::max(max_w, extent(s));
    PassPlan& pp = backward ? g.bwd : g.fwd;
    const int kmax = std::max(max_h, max_w);
    int k0 = 1;
    if (o.max_subtile > 0) k0 = std::max(1, (kmax + o.max_subtile - 1) / o.max_subtile);
    auto try_split = [&](int ky, int kx) -> size_t {       // bytes if it fits, else 0
        build_axis(pp.y, ay, g.tile_y, ky);
        build_axis(pp.x, ax, g.tile_x, kx);
        size_t bytes;
        if (o.tensor_cores) bytes = backward ? layout_backward_tc(g, pp.y, pp.x, pp.stages) : layout_forward_tc(g, pp.y, pp.x, pp.stages);
        else bytes = backward ? layout_backward(g, pp.y, pp.x, pp.dz_ch) : layout_forward(g, pp.y, pp.x);
        size_t budget = (size_t)o.smem_bytes;
        if (o.tensor_cores) budget = std::min<size_t>(pp.ctas == 2 ? kTcSmemBudget2 : kTcSmemBudget, (size_t)o.smem_bytes + 2048);
        return bytes <= budget ? bytes : 0;
    };
    for (int k = k0; k <= kmax; ++k) {
        const int cand[3][2] = {{k, k}, {k + 1, k}, {k, k + 1}};
        for (const auto& c : cand) {
            const int ky = std::min(c[0], max_h), kx = std::min(c[1], max_w);
            size_t bytes = try_split(ky, kx);
            if (!bytes) continue;
            if (backward || o.max_subtile > 0) { pp.smem_bytes = bytes; return FTP_OK; }
            if (o.tensor_cores) {
                // tensor-core stacks: per-stack overheads outweigh a fuller last round, but with fewer stacks
                // than blocks that can run at once a finer split puts the idle SMs to work
                const int slots = kSmCount * pp.ctas;
                int best_ky = ky, best_kx = kx, best_items = N * pp.y.count * pp.x.count;
                if (best_items < slots)
                    for (int dy = 0; dy <= 3; ++dy)
                        for (int dx = 0; dx <= 3; ++dx) {
                            const int yy = std::min(ky + dy, max_h), xx = std::min(kx + dx, max_w);
                            if (!try_split(yy, xx)) continue;
                            const int items = N * pp.y.count * pp.x.count;
                            if (items <= slots && items > best_items) { best_items = items; best_ky = yy; best_kx = xx; }
                        }
                pp.smem_bytes = try_split(best_ky, best_kx);
                return FTP_OK;
            }
            // forward: look a little further for a split that wastes less of the last round
            int best_ky = ky, best_kx = kx;
            double best = -1, fixed = 0;     // fixed: per-stack cost that does not shrink with the tile (loads, syncs)
            for (int dy = 0; dy <= 3; ++dy)
                for (int dx = 0; dx <= 3; ++dx) {
                    const int yy = std::min(ky + dy, max_h), xx = std::min(kx + dx, max_w);
                    if (!try_split(yy, xx)) continue;
                    double done = 0, untiled = 0;
                    count_macs(g, pp, &done, &untiled);
                    const double items = (double)N * pp.y.count * pp.x.count;
                    const double slots = (double)kSmCount * pp.ctas;
                    const double rounds = std::ceil(items / slots);
                    if (dy == 0 && dx == 0) fixed = 0.3 * done * N / items;
                    const double est = rounds * (done * N / items + fixed);
                    if (best < 0 || est < best * 0.97) { best = est; best_ky = yy; best_kx = xx; }
                }
            pp.smem_bytes = try_split(best_ky, best_kx);
            return FTP_OK;
        }
    }
    return FTP_ERR_WORKSPACE;
}

// Multiply-accumulates of the sub-tile stacks of one pass (halo recomputation included) and of the
// untiled layers.
void count_macs(const GroupPlan& g, const PassPlan& pp, double* done, double* untiled)
{
    *done = 0; *untiled = 0;
    for (int i = 0; i < g.n_ops; ++i) {
        const OpDesc& op = g.fwd_ops[i];
        if (op.kind == kOpPool) continue;
        const double f = op.kind == kOpConvPool ? 2.0 : 1.0;     // conv runs at twice the pooled extent
        const double per_px = (double)op.cin * op.cout * op.k * op.k;
        const AxisTables& ty = pp.y; const AxisTables& tx = pp.x;
        double sy = 0, sx = 0;
        for (int r = 0; r < ty.count; ++r)
            sy += f * (ty.span[((size_t)(i + 1) * ty.count + r) * 2 + 1] - ty.span[((size_t)(i + 1) * ty.count + r) * 2] + 1);
        for (int q = 0; q < tx.count; ++q)
            sx += f * (tx.span[((size_t)(i + 1) * tx.count + q) * 2 + 1] - tx.span[((size_t)(i + 1) * tx.count + q) * 2] + 1);
        *done += per_px * sy * sx;
        *untiled += per_px * (f * op.out_H) * (f * op.out_W);
    }
}

// ---- cost terms of one pass of an executed group ----
// Work on the critical path of one pass: every term is the total over all sub-tile stacks of the
// pass divided by the number of stacks that run side by side (blocks in flight; in the backward
// pass the busiest block decides).  The planner's estimate of the pass time is a
// weighted sum of the terms (see kCostWeights).  Terms, fp32 path (multiply-accumulates in units of
// 1e6, bytes in MB, elements in units of 1e6):
//   forward : 0 conv MACs, 1 conv+pool MACs, 2 filter MB read, 3 map MB read + written, 4 ops, 5 outputs, 7 one launch
//   backward: 0 filter-gradient MACs, 1 input-delta MACs of convs, 2 of conv+pool ops, 3 filter MB read,
//             4 partial-set MB updated, 5 map MB, 6 ops, 7 one launch
// bf16 path (tensor-core time in units of 1e3 cycles, taking an MMA with N accumulator columns as max(45, N/2)):
//   forward : 0 MMA cycles, 1 elements of the fp32 network input, 2 filter MB streamed (once per round of accumulators),
//             3 map MB, 4 ops, 5 accumulator elements read back, 6 of these, the ones that go through a fused pool
//   backward: 0 filter-gradient MMA cycles, 1 input-delta MMA cycles, 3 filter MB, 4 partial-set MB, 5 map MB, 6 ops
constexpr int kCostMaxConvs = 3;   // conv layers per executed group the cost model considers (what the weights were fitted on)
inline double mma_cycles(int n) { return n <= 0 ? 0.0 : std::max(45.0, n / 2.0); }

void pass_cost_terms(const ftp_plan& p, const GroupPlan& g, bool backward, bool need_dx, double f[kCostTerms])
{
    for (int k = 0; k < kCostTerms; ++k) f[k] = 0;
    const bool tcp = p.precision == FTP_BF16_FP32ACC;
    const PassPlan& pp = backward ? g.bwd : g.fwd;
    const AxisTables& ty = pp.y; const AxisTables& tx = pp.x;
    const int N = p.N, n = g.n_ops;
    const int tmem_cols = kTcTmemCols / std::max(1, pp.ctas);
    auto ext = [](const AxisTables& t, int m, int r) { return t.span[((size_t)m * t.count + r) * 2 + 1] - t.span[((size_t)m * t.count + r) * 2] + 1; };
    auto own = [](const AxisTables& t, int m, int r) { return t.cell[((size_t)m * t.count + r) * 2 + 1] - t.cell[((size_t)m * t.count + r) * 2] + 1; };
    const double param_mb = g.param_floats * 4.0 / 1e6;
    const int in_bytes = tcp && g.first > 1 ? 2 : 4, out_bytes = tcp ? 2 : 4;
    for (int r = 0; r < ty.count; ++r)
        for (int q = 0; q < tx.count; ++q) {
            // one sub-tile stack (one image); all terms are multiplied by N at the end
            for (int i = 0; i < n; ++i) {
                const OpDesc& op = g.fwd_ops[i];
                const int oh = ext(ty, i + 1, r), ow = ext(tx, i + 1, q);       // output span of the op
                const int ih = ext(ty, i, r), iw = ext(tx, i, q);               // input span
                const int cin_b = tcp ? op.cin16 : op.cin, cout_b = tcp ? op.cout16 : op.cout;
                if (backward) f[5] += (double)cin_b * ih * iw * (tcp ? 2 : 4) / 1e6;   // copy of the op's input
                if (backward) f[6] += 1; else f[4] += 1;
                if (op.kind == kOpPool) continue;
                const int coh = op.S * oh, cow = op.S * ow;                     // conv output span
                const double macs = (double)coh * cow * op.cin * op.cout * op.k * op.k / 1e6;
                const double w_mb = tcp ? (double)op.k * op.k * op.cin16 * op.cout16 * 2 / 1e6
                                        : (double)op.k * op.k * op.cin * op.cout * 4 / 1e6;
                const bool dx = backward && (need_dx || i > 0);
                if (!tcp) {
                    // the direct convolutions give every thread 4 rows x 8 channels of one output column and
                    // run in rounds of kThreads such tasks: count the multiply-accumulates of full rounds
                    auto conv_macs = [&](int rows, int cols, int co_pad, int ci) {
                        const long long tasks = (long long)(co_pad / kCoutTile) * ((rows + 3) / 4) * cols;
                        return (double)((tasks + kThreads - 1) / kThreads) * kThreads * 4 * kCoutTile * ci * op.k * op.k / 1e6;
                    };
                    if (!backward) {
                        f[op.kind == kOpConvPool ? 1 : 0] += conv_macs(coh, cow, op.cout_pad, op.cin);
                        f[2] += w_mb;
                        f[5] += (double)coh * cow * op.cout / 1e6;
                    } else {
                        f[0] += macs;
                        if (dx) {
                            f[op.kind == kOpConvPool ? 2 : 1] += conv_macs(ih, iw, op.cin_pad, op.cout);
                            f[3] += w_mb;
                        }
                    }
                } else if (!backward) {
                    const int nblocks = ((coh + 15) / 16) * ((cow + 7) / 8);
                    const int at_once = std::max(1, tmem_cols / op.cout16);
                    const int rounds = (nblocks + at_once - 1) / at_once;
                    const double per_block = (double)op.k * op.k * (op.cin16 / 16) *
                                             (mma_cycles(std::min(op.cout16, 256)) + mma_cycles(op.cout16 - 256));
                    f[0] += nblocks * per_block / 1e3;
                    f[2] += rounds * w_mb;
                    f[5] += (double)nblocks * 128 * op.cout16 / 1e6;
                    if (op.kind == kOpConvPool) f[6] += (double)coh * cow * op.cout16 / 1e6;
                } else {
                    const int Wp = cow + 2 * (op.k - 1);
                    const int nk = ((coh - 1) * Wp + cow + 15) / 16;
                    const int slices = op.cout16 <= 64 ? 1 : (op.cout16 + 127) / 128;
                    const bool folded = op.cin <= 8;
                    const int units = folded ? op.k : op.k * op.k;
                    const int ucols = folded ? (8 * op.k + 15) / 16 * 16 : op.cin16;
                    f[0] += (double)slices * nk * (units * (mma_cycles(std::min(ucols, 256)) + mma_cycles(ucols - 256)) + 45.0) / 1e3;
                    if (dx) {
                        const int nblocks = ((ih + 15) / 16) * ((iw + 7) / 8);
                        const int at_once = std::max(1, tmem_cols / op.cin16);
                        const int rounds = (nblocks + at_once - 1) / at_once;
                        f[1] += (double)nblocks * op.k * op.k * (op.cout16 / 16) *
                                (mma_cycles(std::min(op.cin16, 256)) + mma_cycles(op.cin16 - 256)) / 1e3;
                        f[3] += rounds * w_mb;
                    }
                }
                (void)cin_b; (void)cout_b;
            }
            // maps read and written in global memory by the stack
            const OpDesc& o0 = g.fwd_ops[0]; const OpDesc& ol = g.fwd_ops[n - 1];
            const double in_mb = (double)(tcp ? o0.cin16 : o0.cin) * ext(ty, 0, r) * ext(tx, 0, q) / 1e6;
            const double out_mb = (double)(tcp ? ol.cout16 : ol.cout) * own(ty, n, r) * own(tx, n, q) / 1e6;
            if (!backward) {
                f[3] += in_mb * in_bytes;
                if (tcp && g.first == 1) f[1] += (double)o0.cin * ext(ty, 0, r) * ext(tx, 0, q) / 1e6;
                for (int i = 0; i < n; ++i) {                                  // every op's output map is kept for the backward pass
                    const OpDesc& op = g.fwd_ops[i];
                    f[3] += (double)(tcp ? op.cout16 : op.cout) * own(ty, i + 1, r) * own(tx, i + 1, q) * out_bytes / 1e6;
                }
            } else {
                f[5] += out_mb * out_bytes;                                    // delta at the group's output
                if (need_dx) f[5] += in_mb * 4 * 2;                            // per-stack input delta, written then summed
                f[4] += param_mb;
            }
        }
    // stacks that run side by side
    double parallel;
    const double items = (double)N * ty.count * tx.count;
    if (!backward) {
        const double slots = (double)kSmCount * pp.ctas;
        parallel = items / std::ceil(items / slots);
    } else {
        const long long busiest = ((long long)items + pp.blocks - 1) / pp.blocks;       // stacks of the busiest block
        parallel = items / busiest;
    }
    for (int k = 0; k < kCostTerms - 1; ++k) f[k] = f[k] * N / parallel;
    f[kCostTerms - 1] = 1.0;
}

// Microseconds per unit of each term, fitted (non-negative least squares on relative errors) to the
// kernel times of 168 candidate groups per precision, each measured inside whole training steps of
// the 8- and 16-layer stacks on one B200 (calibrate.py of the Python package measures them and prints
// this table).  Error of the fit, |log(estimate / measured)|: median 0.04-0.06, 90th percentile
// 0.13-0.23 over the four (precision, pass) fits.
const double kCostWeights[2][2][kCostTerms] = {
    {   // fp32: forward, backward
        {6.444, 7.033, 18.79, 143.4, 5.824, 34.41, 0, 7.93},
        {10.61, 3.967, 2.645, 274.6, 0, 261.3, 37.98, 5.55},
    },
    {   // bf16
        {0, 1360, 34.42, 32.26, 3.056, 91.07, 229.4, 8.708},
        {0.4465, 1.076, 0, 0, 78.93, 59.32, 6.233, 14.05},
    },
};

double pass_estimate_us(int precision, bool backward, const double f[kCostTerms])
{
    const double* w = kCostWeights[precision == FTP_BF16_FP32ACC ? 1 : 0][backward ? 1 : 0];
    double t = 0;
    for (int k = 0; k < kCostTerms; ++k) t += w[k] * f[k];
    return t;
}

// Weight-stationary groups: multiply-accumulates at the measured rate of the kernels, the maps they move
// at HBM speed, one launch overhead per kernel.
double stationary_estimate_us(const ftp_plan& p, const GroupPlan& g, bool backward, bool need_dx)
{
    const OpDesc& op = g.fwd_ops[0];
    const double px = (double)p.N * op.in_H * op.in_W;
    const double flops = 2.0 * px * op.cin * op.cout * op.k * op.k;
    const double rate = (op.k == 1 || g.st.thin ? kStatTflops1x1 : kStatTflops) * 1e6;   // flop per microsecond
    const double map_us = px * (op.cin + op.cout) * 4.0 / 6.5e6;                   // bytes at 6.5 TB/s
    if (!backward) return flops / rate + map_us + 5.0;
    return flops * (need_dx ? 2.0 : 1.0) / rate + 3.0 * map_us + 15.0;
}

// One-conv groups of the bf16 path (banded convolutions, weight-stationary filter gradient): padded multiply-
// accumulates at the rates measured for the kernels on B200 (convolutions: about 800 TFLOP/s with slices of 80 channels
// and more, in proportion below that, since a narrow MMA costs the tensor core about as much as a wide one; filter
// gradient: 600), the maps at 5 TB/s, a few microseconds a launch.
double tc_stationary_estimate_us(const ftp_plan& p, const GroupPlan& g, bool backward, bool need_dx)
{
    const OpDesc& op = g.fwd_ops[0];
    const double px = (double)p.N * op.in_H * op.in_W;
    const int cin16 = g.col_cin16 ? g.col_cin16 : op.cin16, kk = g.col_cin16 ? 1 : op.k * op.k;
    const double flops = 2.0 * px * cin16 * op.cout16 * kk;
    auto rate = [](int ns) { return 800e6 * std::min(1.0, std::max(ns, 16) / 80.0); };           // flop per microsecond
    const double in_b = px * cin16 * 2.0, out_b = px * op.cout16 * 2.0 / (op.kind == kOpConvPool ? 4.0 : 1.0), dz_b = px * op.cout16 * 2.0;
    if (!backward) return flops / rate(g.cf.Ns) + (in_b + out_b) / 5e6 + (g.col_cin16 ? in_b / 3e6 : 0.0) + 8.0;
    double t = (2.0 * out_b + dz_b) / 5e6 + 4.0;                                               // dz planes
    t += flops / 600e6 + (in_b + dz_b) / 5e6 + 10.0;                                           // filter gradient
    if (need_dx) t += flops / rate(g.cd.Ns) + (in_b + dz_b) / 5e6 + (g.col_cin16 ? in_b / 3e6 : 0.0) + 8.0;
    return t;
}

// Backward launch shape: as many blocks as run at once (or as there are stacks), each owning one
// partial gradient set; the stacks of the whole batch are dealt out evenly to them.
void set_backward_blocks(GroupPlan& g, int N, int gy, int gx)
{
    (void)gy; (void)gx;
    const long long items = (long long)N * g.bwd.y.count * g.bwd.x.count;
    g.bwd.blocks = (int)std::max<long long>(1, std::min<long long>(items, (long long)kSmCount * g.bwd.ctas));
}

// Backward sub-tiling, second step.  choose_subtiles takes the largest sub-tiles that fit; the
// blocks then share the N x (sub-tiles of the map) stacks, and when that number does not divide by
// the blocks the slowest block runs one stack more than the average.  A somewhat finer split can
// even that out (296 stacks of 1/8 tile on 148 blocks beat 216 stacks of 1/6).  The
// candidates up to three cuts finer per axis are compared by the time model's estimate of the
// pass, which counts the stacks of the busiest block; the first split stays unless another is
// estimated at least 3 % faster.
void refine_backward_split(const ftp_plan& p, GroupPlan& g, const PlanOpts& o)
{
    PassPlan& pp = g.bwd;
    const AxisInfo ay = axis_info(g, true), ax = axis_info(g, false);
    int max_h = 0, max_w = 0, ky0 = 1, kx0 = 1;
    for (const Span& s : g.tile_y) max_h = std::max(max_h, extent(s));
    for (const Span& s : g.tile_x) max_w = std::max(max_w, extent(s));
    for (size_t t = 0; t + 1 < pp.y.tile_begin.size(); ++t) ky0 = std::max(ky0, pp.y.tile_begin[t + 1] - pp.y.tile_begin[t]);
    for (size_t t = 0; t + 1 < pp.x.tile_begin.size(); ++t) kx0 = std::max(kx0, pp.x.tile_begin[t + 1] - pp.x.tile_begin[t]);
    size_t budget = (size_t)o.smem_bytes;
    if (o.tensor_cores) budget = std::min<size_t>(pp.ctas == 2 ? kTcSmemBudget2 : kTcSmemBudget, (size_t)o.smem_bytes + 2048);
    auto eval = [&](int ky, int kx) -> double {               // estimate in microseconds, negative if it does not fit
        build_axis(pp.y, ay, g.tile_y, ky);
        build_axis(pp.x, ax, g.tile_x, kx);
        const size_t bytes = o.tensor_cores ? layout_backward_tc(g, pp.y, pp.x, pp.stages) : layout_backward(g, pp.y, pp.x, 0);
        if (bytes > budget) return -1.0;
        pp.smem_bytes = bytes;
        set_backward_blocks(g, p.N, p.grid_y, p.grid_x);
        double f[kCostTerms];
        pass_cost_terms(p, g, true, g.first > 1, f);
        return pass_estimate_us(p.precision, true, f);
    };
    const double first = eval(ky0, kx0);
    double best = first;
    int best_ky = ky0, best_kx = kx0;
    if (first > 0)
        for (int dy = 0; dy <= 3; ++dy)
            for (int dx = 0; dx <= 3; ++dx) {
                if (!dy && !dx) continue;
                const int ky = std::min(ky0 + dy, max_h), kx = std::min(kx0 + dx, max_w);
                const double est = eval(ky, kx);
                if (est > 0 && est < 0.97 * first && est < best) { best = est; best_ky = ky; best_kx = kx; }
            }
    eval(best_ky, best_kx);
}

// Weight-stationary execution of a group that holds one conv layer (optionally with its pool), fp32
// path: launch shapes of the three kernels.  The convolution cuts (row pairs of the whole batch) x
// (columns) x (output channels) into blocks of 16 x 8 x 64; the filter gradient gives every 64 x 32
// slice of (output, input) channels `fg_splits` blocks, each with an equal share of the pixel stages
// and one partial set, so that about two rounds of blocks fill the GPU.
void plan_stationary(const ftp_plan& p, GroupPlan& g, const PlanOpts& o)
{
    g.st = StatPlan{};
    if (p.precision != FTP_FP32 || o.stationary < 0 || g.n_ops != 1) return;
    const OpDesc& op = g.fwd_ops[0];
    if (op.kind == kOpPool || (op.k != 1 && op.k != 3)) return;
    const bool thin = op.kind == kOpConvPool && op.k == 3 && op.cin <= 4 && op.cout <= 32;
    if (o.stationary == 0 && op.cin < kStatMinCin && !thin) return;
    const int H = op.in_H, W = op.in_W;                        // the conv's resolution
    const long long rp_total = (long long)p.N * ((H + 1) / 2);
    const int x_tiles = (W + kStCols - 1) / kStCols;
    // blocks of 64 output channels x 16 row pairs, or of 32 x 32 where that wastes fewer channels or rows, i.e. takes
    // fewer rounds of blocks (two blocks run per SM)
    auto conv_blocks = [&](int cout, int ct, int threads = kStThreads) {
        const int rpt = st_row_pairs(ct, threads);
        return (rp_total + rpt - 1) / rpt * x_tiles * ((cout + ct - 1) / ct);
    };
    // Blocks of 128 threads (half the row pairs, four per SM) where whole blocks fill less than a round and a half of
    // the 2 x 148 slots: the SMs that get one block more than the others then wait for half a block, not a whole one
    // (measured on C1, batch 4: 10-18 % on such launches; with more rounds, or with a contraction over 512 channels x 9
    // window positions, where C3's 38 x 38 input deltas lost 10 %, the shorter stages cost more than the finer split saves).
    auto pick_threads = [&](long long blocks256, int depth) {
        return blocks256 <= 3LL * kSmCount && depth <= 2304 ? 128 : kStThreads;
    };
    auto pick_tile = [&](int cout) {
        if (cout <= 32) return 32;
        const long long slots = 2LL * kSmCount;
        // both shapes do the same work per block (64 x 16 or 32 x 32 thread tiles): what differs is how many
        // blocks the padded channel and row counts give, i.e. how many rounds of `slots` blocks
        const long long r64 = (conv_blocks(cout, 64) + slots - 1) / slots, r32 = (conv_blocks(cout, 32) + slots - 1) / slots;
        return r32 < r64 ? 32 : 64;
    };
    const int fwd_ct = pick_tile(op.cout), dx_ct = pick_tile(op.cin);
    const int fwd_thr = o.stationary == 1 ? kStThreads : pick_threads(conv_blocks(op.cout, fwd_ct), op.cin * op.k * op.k);
    const int dx_thr = o.stationary == 1 ? kStThreads : pick_threads(conv_blocks(op.cin, dx_ct), op.cout * op.k * op.k);
    const long long fwd_blocks = conv_blocks(op.cout, fwd_ct, fwd_thr), dx_blocks = conv_blocks(op.cin, dx_ct, dx_thr);
    // filter gradient: 3 x 3 in stages of 4 row pairs x 8 columns and 64 x 32 channel slices; 1 x 1 as a contraction over
    // stages of 32 flat pixels of an image and 64 x 128 channel slices
    const long long stages = op.k == 1 ? (long long)p.N * ((H * W + kFg1Px - 1) / kFg1Px)
                                       : (rp_total + kFgRowPairs - 1) / kFgRowPairs * x_tiles;
    const long long slices = op.k == 1 ? (long long)((op.cout + kFg1Co - 1) / kFg1Co) * ((op.cin + kFg1Ci - 1) / kFg1Ci)
                                       : (long long)((op.cout + kFgCo - 1) / kFgCo) * ((op.cin + kFgCi - 1) / kFgCi);
    if (fwd_blocks > 0x7fffffffLL || dx_blocks > 0x7fffffffLL || stages > 0x7fffffffLL || slices > 65535) return;
    g.st.on = 1; g.st.k = op.k; g.st.pool = op.kind == kOpConvPool ? 1 : 0;
    g.st.fwd_blocks = (int)fwd_blocks; g.st.dx_blocks = (int)dx_blocks;
    g.st.fwd_co_tile = fwd_ct; g.st.dx_co_tile = dx_ct;
    g.st.fwd_threads = fwd_thr; g.st.dx_threads = dx_thr;
    g.st.fg_stages = (int)stages;
    // one round of the blocks that run at once (2 per SM; 1 x 1: 3): the input-delta convolution on the other stream fills
    // what a round leaves idle, and every share costs a partial set that the reduction has to read; at least 4 stages a share
    const long long slots = (op.k == 1 ? 3LL : 2LL) * kSmCount;
    g.st.fg_splits = (int)std::max<long long>(1, std::min<long long>(std::max<long long>(1, stages / 4), slots / slices));
    g.st.fg_blocks = (int)(slices * g.st.fg_splits);
    g.bwd.blocks = g.st.fg_splits;                             // partial gradient sets of the group
    g.bwd.scratch_floats = 0;                                  // the input delta is written whole, no overlapping parts to sum
    if (thin && o.stationary <= 0) {                           // (stationary = 1 forces the general kernels, for tests)
        g.st.thin = 1;
        g.st.thin_tiles_y = (op.out_H + kThinTileH - 1) / kThinTileH;
        g.st.thin_tiles_x = (op.out_W + kThinTileW - 1) / kThinTileW;
        const long long tiles = (long long)p.N * g.st.thin_tiles_y * g.st.thin_tiles_x;
        g.st.thin_blocks = (int)std::min<long long>(tiles, 2LL * kSmCount);
        g.bwd.blocks = g.st.thin_blocks;                       // one partial set per block
    }
}

// bf16 path: whether a conv layer runs as a group of its own with the weight-stationary filter gradient: window 1
// or 3, rows of at most 256 tile entries, a saved bf16 map as input, i.e. not the first layer.  (Measured on B200
// this beats the fused sub-tile stacks for every such layer of the YOLO stacks, by 2x to 6x for the backward pass of
// the layers with 128 channels and more, whose per-sub-tile gradient flush it removes.)
bool tc_stationary_conv(const ftp_plan& p, int li /*0-based*/, const PlanOpts& o)
{
    const ftp_layer& l = p.layers[li];
    if (p.precision != FTP_BF16_FP32ACC || o.stationary < 0 || l.kind != FTP_CONV) return false;
    // the first layer reads the fp32 network input: only as a 1x1 conv on its window-unrolled copy (3x3, at most 7 channels)
    if (li == 0 && (l.k != 3 || l.cin * 9 > 64)) return false;
    return (l.k == 1 || l.k == 3) && p.maps[li].W <= kTcMaxColChunks * 126;
}

// Column chunks of a band: as few as keep the tile pitch (chunk + k - 1) within the 128 pixels of a TMA box row,
// of equal (even) width.
void tc_col_chunks(int W, int* ncc, int* Cw)
{
    *ncc = (W + 125) / 126;
    *Cw = ((W + *ncc - 1) / *ncc + 1) / 2 * 2;
    if (*Cw > W) *Cw = W;
}

// Launch shape of the banded convolution kernel for a conv with `cout16` output and `cin16` input channels (padded)
// on N maps of H x W: bands as tall as the accumulators allow (512 columns = blocks of 128 entries x Ns channels),
// among those the height with the fewest rounds of blocks over the SMs; as many stages as fit.
TcConvPlan plan_tc_conv_kpc(int N, int H, int W, int K, int cin16, int cout16, bool pool, int kpc3);

TcConvPlan plan_tc_conv(int N, int H, int W, int K, int cin16, int cout16, bool pool)
{
    // input channels per chunk: 3x3: 16, or 32 with slices of at most 64 channels where two stages of that size fit
    // (their filters are small, and every chunk costs the issuers a wait, a fence and a commit); 1x1: up to 64
    if (K == 3 && std::min(cout16, 128) <= 64 && cin16 >= 32) {
        const TcConvPlan c = plan_tc_conv_kpc(N, H, W, K, cin16, cout16, pool, 4);
        if (c.on) return c;
    }
    return plan_tc_conv_kpc(N, H, W, K, cin16, cout16, pool, 2);
}

TcConvPlan plan_tc_conv_kpc(int N, int H, int W, int K, int cin16, int cout16, bool pool, int kpc3)
{
    TcConvPlan c;
    tc_col_chunks(W, &c.ncc, &c.Cw);
    c.Wp = c.Cw + K - 1;
    c.Ns = std::min(cout16, 128);
    c.slices = (cout16 + c.Ns - 1) / c.Ns;
    // slices of at most 64 channels: items of 256 columns in two alternating buffers (narrow MMAs leave the tensor
    // core idle while an item is read back); wider slices: one buffer of 512 columns (their filters are read per item)
    c.nbuf = c.Ns <= 64 ? 2 : 1;
    const int max_blk = std::min(8, kTcTmemCols / c.nbuf / c.Ns);
    c.kpc = K == 1 ? std::min(cin16 / 8, 8) : kpc3;
    const int step = pool ? 2 : 1;
    const int r_max = std::min((max_blk * 128) / c.Wp, H) / step * step;
    if (r_max < step) return c;
    double best = -1;
    for (int R = step; R <= r_max; R += step) {
        const int bands = (H + R - 1) / R * c.ncc, nblk = (R * c.Wp + 127) / 128;
        const long long items = (long long)N * bands * c.slices;
        const double cost = (double)((items + kSmCount - 1) / kSmCount) * (nblk + 0.5);      // rounds x (MMAs + fixed part) of a block
        if (best < 0 || cost <= best) { best = cost; c.R = R; c.nblk = nblk; c.bands_img = bands; }
    }
    const size_t entries = std::max<size_t>((size_t)(c.R + K - 1) * c.Wp, (size_t)c.nblk * 128 + (size_t)(K - 1) * c.Wp + K);
    c.x_plane = (int)align_up(entries * 16, 128);
    c.stage_bytes = c.kpc * c.x_plane + K * K * c.kpc * c.Ns * 16;
    // fused pool: the band as stored goes through a staging area, all channels of the slice at once where that leaves
    // three stages (two for short rings), else 16 channels or more at a time
    const size_t room = (size_t)kTcConvSmemBudget - kTcFgHeader;
    const size_t plane_pair = (size_t)c.nblk * 128 * 16 * 2, whole = (size_t)(c.Ns / 16) * plane_pair;
    size_t staging = pool ? kTcPoolStageBytes : 0;
    c.stages = (int)std::min<size_t>(4, (room - staging) / c.stage_bytes);
    if (pool) {
        const int keep = std::min(c.stages, 3);
        if (room >= (size_t)keep * c.stage_bytes + whole) { c.stages = std::min<int>(c.stages, (int)((room - whole) / c.stage_bytes)); staging = whole; }
        else staging = std::max<size_t>(staging, (room - (size_t)c.stages * c.stage_bytes) / plane_pair * plane_pair);
        c.pool_planes = (int)(staging / plane_pair) * 2;
        c.pool_stage_bytes = (int)staging;
    }
    if (c.stages < 2 || (pool && c.pool_planes < 2)) return c;
    c.smem_bytes = kTcFgHeader + c.stages * c.stage_bytes + (int)staging;
    const long long items = (long long)N * c.bands_img * c.slices;
    if (items > 0x7fffffffLL) return c;
    c.items = (int)items;
    c.blocks = (int)std::min<long long>(items, kSmCount);
    c.on = 1;
    return c;
}

// Launch shape of the weight-stationary filter gradient of a one-conv bf16 group (tc_stationary.cuh): slices of
// Ms output x ncols input channels (all window positions of a slice fit the 512 tensor-memory columns), bands of
// R rows chosen for the fewest K steps among those whose two stages fit in shared memory, and as many pixel
// shares as fill the SMs once.
void plan_tc_filter_grad(const ftp_plan& p, GroupPlan& g, const PlanOpts& o)
{
    g.tfg = TcFgPlan{};
    if (g.n_ops != 1 || g.bwd_ops[0].kind == kOpPool || !tc_stationary_conv(p, g.first - 1, o)) return;
    const OpDesc& op = g.bwd_ops[0];
    TcFgPlan t;
    const bool unrolled = g.first == 1;                         // first layer: 1x1 conv on the window-unrolled input
    const int col_cin16 = round_up(op.cin * 9, 16);
    const int H = op.in_H, W = op.in_W, K = unrolled ? 1 : op.k;
    const int cin16 = unrolled ? col_cin16 : op.cin16;
    tc_col_chunks(W, &t.ncc, &t.Cw);
    t.k = K; t.Wp = t.Cw + K - 1;
    t.Ms = op.cout16 <= 64 ? 64 : 128;
    t.slices = (op.cout16 + t.Ms - 1) / t.Ms;
    t.ncols = std::min(cin16, K == 1 ? 256 : 48);
    if (K == 3 && cin16 > 32) {
        // 48 or 32 input channels a block: the slowest block sets the time, i.e. rounds of blocks over the SMs x the pixels
        // of a share x the cycles of an MMA that wide (32 + columns / 4: both operands come from shared memory).  32 wins
        // where 48 leaves a ragged last slice as wide (64 = 48 + 16 against 32 + 32) or too few blocks for the SMs
        // (512 -> 1024: 88 blocks against 128)
        double best_cost = -1;
        for (int nc : {48, 32}) {
            const long long roles = (long long)t.slices * ((cin16 + nc - 1) / nc);
            const long long shares = std::max<long long>(1, kSmCount / roles);
            const double cost = (double)((roles * shares + kSmCount - 1) / kSmCount) / (double)shares * (32.0 + nc / 4.0);
            if (best_cost < 0 || cost < best_cost) { best_cost = cost; t.ncols = nc; }
        }
    }
    t.nci = (cin16 + t.ncols - 1) / t.ncols;
    long long best = -1;
    for (int R = 1; R <= std::min(H, 64); ++R) {
        const size_t dzp = align_up(((size_t)R * t.Wp + 16) * 16, 128), xp = align_up(((size_t)(R + K - 1) * t.Wp + 32) * 16, 128);
        const size_t stage = (size_t)(t.Ms / 8) * dzp + (size_t)(t.ncols / 8) * xp;
        if (kTcFgHeader + 2 * stage > (size_t)kTcFgSmemBudget || R + K - 1 > 256) break;
        const long long cost = (long long)((H + R - 1) / R) * ((R * t.Wp + 15) / 16 * 16 + 32);
        if (best < 0 || cost <= best) {
            best = cost; t.R = R; t.dz_plane = (int)dzp; t.x_plane = (int)xp; t.stage_bytes = (int)stage;
        }
    }
    if (best < 0) return;
    t.smem_bytes = kTcFgHeader + 2 * t.stage_bytes;
    t.bands_img = (H + t.R - 1) / t.R * t.ncc;
    const long long bands = (long long)p.N * t.bands_img;
    if (bands > 0x7fffffffLL) return;
    t.bands = (int)bands;
    const int roles = t.slices * t.nci;
    t.shares = (int)std::max<long long>(1, std::min<long long>(bands, kSmCount / roles));
    t.blocks = roles * t.shares;
    // the forward convolution, and the input delta as the convolution of dz (cout16 channels) with the rotated filters
    g.cf = plan_tc_conv(p.N, H, W, K, cin16, op.cout16, op.kind == kOpConvPool);
    g.cd = plan_tc_conv(p.N, H, W, K, op.cout16, cin16, false);
    if (!g.cf.on || !g.cd.on) return;
    if (unrolled) { g.col_cin = op.cin * 9; g.col_cin16 = col_cin16; }
    t.on = 1;
    g.tfg = t;
    g.bwd.scratch_floats = 0;       // no per-sub-tile input deltas
}

struct LayerOffsets { std::vector<long long> p_off, wf_off, wb_off, twf_off, twb_off; };

// Builds the ops, the sub-tiling and the block counts of one executed group (layers first..last).
// Returns FTP_ERR_WORKSPACE if nothing fits; *redundancy is the larger of the two passes' ratios of
// multiply-accumulates executed to untiled ones.
int make_group(const ftp_plan& p, const LayerOffsets& lo, int first, int last, const PlanOpts& o, GroupPlan& g,
               double* redundancy)
{
    g = GroupPlan{};
    g.first = first; g.last = last;
    const int N = p.N, gy = p.grid_y, gx = p.grid_x;
    const MapShape& out = p.maps[last];
    g.tile_y = equal_partition(0, out.H, gy);
    g.tile_x = equal_partition(0, out.W, gx);
    g.param_begin = -1;
    long long gp = 0, tgp = 0;
    const bool tcp = p.precision == FTP_BF16_FP32ACC;
    for (int li = first - 1; li < last; ++li) {
        const ftp_layer& l = p.layers[li];
        OpDesc op{};
        const bool fuse = l.kind == FTP_CONV && li + 1 < last && p.layers[li + 1].kind == FTP_MAXPOOL;
        const int le = fuse ? li + 1 : li;          // last layer of this op (0-based)
        op.kind = l.kind == FTP_MAXPOOL ? kOpPool : (fuse ? kOpConvPool : kOpConv);
        op.cin = p.maps[li].C; op.cout = p.maps[le + 1].C;
        op.k = l.k; op.pad = l.pad; op.slope = l.leaky;
        op.S = op.kind == kOpConv ? 1 : 2;
        op.keff = op.kind == kOpConvPool ? l.k + 1 : l.k;
        op.prev_has_act = (g.n_ops > 0 && g.fwd_ops[g.n_ops - 1].kind != kOpPool) ? 1 : 0;
        op.in_map = li + 1; op.out_map = le + 2;
        op.in_H = p.maps[li].H; op.in_W = p.maps[li].W;
        op.out_H = p.maps[le + 1].H; op.out_W = p.maps[le + 1].W;
        op.cin16 = round_up(op.cin, 16); op.cout16 = round_up(op.cout, 16);
        if (l.kind == FTP_CONV) {
            op.twf_off = lo.twf_off[li]; op.twb_off = lo.twb_off[li];
            op.tgp_off = tgp;
            tgp += (long long)l.k * l.k * op.cout16 * op.cin16 + op.cout16;
            op.cout_pad = (l.cout + kCoutTile - 1) / kCoutTile * kCoutTile;
            op.cin_pad = (l.cin + kCoutTile - 1) / kCoutTile * kCoutTile;
            op.wf_off = lo.wf_off[li]; op.wb_off = lo.wb_off[li];
            op.p_off = lo.p_off[li];
            if (g.param_begin < 0) g.param_begin = lo.p_off[li];
            op.gp_off = lo.p_off[li] - g.param_begin;
            gp = op.gp_off + (long long)l.cout * l.cin * l.k * l.k + l.cout;
        }
        g.fwd_ops[g.n_ops] = op;
        g.bwd_ops[g.n_ops] = op;
        ++g.n_ops;
        li = le;
    }
    if (g.param_begin < 0) g.param_begin = 0;
    g.param_floats = (size_t)(tcp ? tgp : gp);

    // Tensor-core path: two blocks per SM hide the latencies of a block's serial phases behind the
    // other block; each then has half of the shared and tensor memory, so no operand of the group may
    // span more than 256 accumulator columns.  Left to the planner, only the forward pass of groups
    // with at most 64 channels runs that way: measured on B200, wider layers and the backward pass
    // (three live tiles) lose more from the smaller sub-tiles than they gain.
    int max_ch = 0;
    for (int i = 0; i < g.n_ops; ++i)
        if (g.fwd_ops[i].kind != kOpPool) max_ch = std::max(max_ch, std::max(g.fwd_ops[i].cin16, g.fwd_ops[i].cout16));
    const int want_fwd = !tcp ? 1 : o.tc_ctas == 0 ? (max_ch <= 64 ? 2 : 1) : (o.tc_ctas == 2 && max_ch <= 256 ? 2 : 1);
    const int want_bwd = tcp && o.tc_ctas == 2 && max_ch <= 256 ? 2 : 1;
    for (int pass = 0; pass < 2; ++pass) {
        PassPlan& pp = pass ? g.bwd : g.fwd;
        pp.ctas = pass ? want_bwd : want_fwd;
        pp.stages = 2;
        int rc = choose_subtiles(g, pass == 1, o, N);
        if (rc != FTP_OK && pp.ctas == 2) { pp.ctas = 1; rc = choose_subtiles(g, pass == 1, o, N); }
        if (rc != FTP_OK) return rc;
        if (pass == 1 && o.max_subtile == 0 && o.refine_backward) refine_backward_split(p, g, o);
        if (pass == 0 && !tcp) {
            // Filter staging: what the chosen sub-tiles leave of the shared memory holds, behind the
            // activation area, two halves of w_ch input channels' filters each (about 32 KB a half at
            // most).  Ops that would get less than kMinFilterStage words per half, unless that is all
            // their filters, read global memory: two barriers per half cost more than short halves save.
            const long long room = ((long long)o.smem_bytes - (long long)pp.smem_bytes) / 4;      // floats
            const int base = (int)((pp.smem_bytes - kSmemHeader) / 4);
            long long used = 0;
            for (int i = 0; i < g.n_ops; ++i) {
                OpDesc& op = g.fwd_ops[i];
                op.w_off = base; op.w_ch = 0;
                if (op.kind == kOpPool) continue;
                const long long per_ci = (long long)op.k * op.k * op.cout_pad;
                long long ch = std::min<long long>(op.cin, std::min<long long>(room / (2 * per_ci), std::max<long long>(2, 8192 / per_ci)));
                if (ch >= 1 && (ch == op.cin || ch * per_ci >= kMinFilterStage)) { op.w_ch = (int)ch; used = std::max(used, 2 * ch * per_ci); }
            }
            pp.smem_bytes += (size_t)used * 4;
        }
        if (pass == 1 && !tcp) {
            // delta staging areas (see layout_backward) where they cost no sub-tile size
            for (int ch : {kDeltaStageChannels, kDeltaStageChannels / 2, kDeltaStageChannels / 4, 0}) {
                pp.dz_ch = ch;
                const size_t bytes = layout_backward(g, pp.y, pp.x, ch);
                if (bytes <= (size_t)o.smem_bytes) { pp.smem_bytes = bytes; break; }
            }
            pp.dz_ch = 0;                                   // report what the ops got
            for (int i = 0; i < g.n_ops; ++i) pp.dz_ch = std::max(pp.dz_ch, g.bwd_ops[i].dz_ch);
            // Staging of the rotated filters for the input-delta convolutions, in what is left: two
            // halves as in the forward pass for a plain conv; for a fused conv+pool with a delta
            // staging area, the filters of its dz_ch channels (all of them or none).
            const long long room = ((long long)o.smem_bytes - (long long)pp.smem_bytes) / 4;
            const int base = (int)((pp.smem_bytes - kSmemHeader) / 4);
            long long used = 0;
            for (int i = 0; i < g.n_ops; ++i) {
                OpDesc& op = g.bwd_ops[i];
                op.w_off = base; op.w_ch = 0;
                if (op.kind == kOpPool) continue;
                const long long per_co = (long long)op.k * op.k * op.cin_pad;
                if (op.kind == kOpConvPool) {
                    if (op.dz_ch > 0 && op.dz_ch * per_co <= room) { op.w_ch = op.dz_ch; used = std::max(used, op.dz_ch * per_co); }
                    continue;
                }
                long long ch = std::min<long long>(op.cout, std::min<long long>(room / (2 * per_co), std::max<long long>(2, 8192 / per_co)));
                if (ch >= 1 && (ch == op.cout || ch * per_co >= kMinFilterStage)) { op.w_ch = (int)ch; used = std::max(used, 2 * ch * per_co); }
            }
            pp.smem_bytes += (size_t)used * 4;
        }
        if (tcp) {
            // a four-stage filter ring where it costs no sub-tile size (measured: paying for it with smaller
            // tiles loses more than the deeper ring gains)
            const size_t budget = std::min<size_t>(pp.ctas == 2 ? kTcSmemBudget2 : kTcSmemBudget, (size_t)o.smem_bytes + 2048);
            const size_t bytes4 = pass ? layout_backward_tc(g, pp.y, pp.x, kTcMaxStages) : layout_forward_tc(g, pp.y, pp.x, kTcMaxStages);
            if (bytes4 <= budget) { pp.stages = kTcMaxStages; pp.smem_bytes = bytes4; }
        }
    }
    double bwd_done = 0, bwd_untiled = 0;
    count_macs(g, g.fwd, &g.macs_done, &g.macs_untiled);
    count_macs(g, g.bwd, &bwd_done, &bwd_untiled);
    if (redundancy)
        *redundancy = g.macs_untiled > 0 ? std::max(g.macs_done, bwd_done) / g.macs_untiled : 1.0;

    g.fwd.blocks = g.fwd.y.count * g.fwd.x.count * N;
    set_backward_blocks(g, N, gy, gx);
    // (tensor-core path, groups after the first: the blocks hold 8-channel planes of the padded channel count)
    g.bwd.scratch_floats = (size_t)N * (tcp && first > 1 ? round_up(p.maps[first - 1].C, 16) : p.maps[first - 1].C) *
                           g.bwd.y.scratch_off[g.bwd.y.count] *
                           g.bwd.x.scratch_off[g.bwd.x.count];
    plan_stationary(p, g, o);
    plan_tc_filter_grad(p, g, o);
    // bf16 path: the fused kernels keep all output channels of an op in the 512 tensor-memory columns; wider layers
    // run on the banded kernels (a group of their own) or not at all
    if (tcp && !g.tfg.on)
        for (int i = 0; i < g.n_ops; ++i)
            if (g.fwd_ops[i].cin > kTcTmemCols || g.fwd_ops[i].cout > kTcTmemCols) return FTP_ERR_LAYERS;
    if (g.st.on) {                                  // no sub-tile stacks, no halo recomputation
        g.macs_done = g.macs_untiled;
        if (redundancy) *redundancy = 1.0;
    }

    return FTP_OK;
}

}  // namespace

int build_plan(ftp_plan& p, const ftp_layer* layers, int n_layers, int N, int C, int H, int W,
               int gy, int gx, const ftp_group* groups, int n_groups, int precision, const PlanOpts& opts)
{
    if (!layers || !groups || n_layers <= 0 || n_groups <= 0 || N <= 0 || C <= 0 || H <= 0 || W <= 0 ||
        gy <= 0 || gx <= 0)
        return FTP_ERR_ARG;
    if (opts.max_redundancy_pct < 100 || opts.max_subtile < 0 || opts.smem_bytes < 2 * kSmemHeader || opts.smem_bytes > kSmemBudget)
        return FTP_ERR_ARG;
    if (precision != FTP_FP32 && precision != FTP_BF16_FP32ACC) return FTP_ERR_ARG;
    const bool tcp = precision == FTP_BF16_FP32ACC;
    PlanOpts popts = opts;
    popts.tensor_cores = tcp ? 1 : 0;
    p.layers.assign(layers, layers + n_layers);
    p.N = N; p.grid_y = gy; p.grid_x = gx; p.precision = precision;
    p.tc_tma = opts.tc_tma < 0 ? 0 : 1;

    // layer validation and map shapes X_1 .. X_{L+1}
    p.maps.clear();
    p.maps.push_back(MapShape{C, H, W});
    LayerOffsets lo;
    lo.p_off.assign(n_layers, 0); lo.wf_off.assign(n_layers, 0); lo.wb_off.assign(n_layers, 0);
    lo.twf_off.assign(n_layers, 0); lo.twb_off.assign(n_layers, 0);
    long long params = 0, wf = 0, wb = 0, twf = 0;
    for (int i = 0; i < n_layers; ++i) {
        const ftp_layer& l = p.layers[i];
        MapShape in = p.maps.back();
        if (l.kind == FTP_CONV) {
            if (l.k < 1 || l.k > 7 || l.k % 2 == 0 || l.stride != 1 || l.pad != l.k / 2 || l.cin != in.C ||
                l.cout <= 0 || !(l.leaky >= 0.0f))
                return FTP_ERR_LAYERS;
            p.maps.push_back(MapShape{l.cout, in.H, in.W});
            lo.p_off[i] = params;
            params += (long long)l.cout * l.cin * l.k * l.k + l.cout;
            int cout_pad = (l.cout + kCoutTile - 1) / kCoutTile * kCoutTile;
            int cin_pad = (l.cin + kCoutTile - 1) / kCoutTile * kCoutTile;
            lo.wf_off[i] = wf; wf += (long long)l.cin * l.k * l.k * cout_pad;
            lo.wb_off[i] = wb; wb += (long long)l.cout * l.k * l.k * cin_pad;
            lo.twf_off[i] = lo.twb_off[i] = twf;        // both packed layouts hold k*k*cin16*cout16 elements; room for the
            twf += (long long)l.k * l.k * round_up(l.cin, 128) * round_up(l.cout, 128);   // banded kernels' padded slices
        } else if (l.kind == FTP_MAXPOOL) {
            if (l.k != 2 || l.stride != 2 || l.pad != 0 || in.H % 2 || in.W % 2) return FTP_ERR_LAYERS;
            p.maps.push_back(MapShape{in.C, in.H / 2, in.W / 2});
        } else {
            return FTP_ERR_LAYERS;
        }
    }
    p.param_floats = (size_t)params;
    p.wf_floats = (size_t)(tcp ? twf : wf);
    p.wb_floats = (size_t)(tcp ? twf : wb);

    // groups: contiguous, covering 1..L
    int expect = 1;
    for (int g = 0; g < n_groups; ++g) {
        if (groups[g].first != expect || groups[g].last < groups[g].first || groups[g].last > n_layers)
            return FTP_ERR_GROUPS;
        expect = groups[g].last + 1;
        const MapShape& out = p.maps[groups[g].last];
        if (gy > out.H || gx > out.W) return FTP_ERR_GRID;
    }
    if (expect != n_layers + 1) return FTP_ERR_GROUPS;
    p.user_groups.assign(groups, groups + n_groups);

    // Executed groups.  A requested group is first cut by the fixed rule: runs of at most
    // max_group_convs conv layers that end with the pool after a conv, shortened further while the halo
    // recomputation exceeds the cap or no sub-tile fits in shared memory.  With the cost model on, all
    // ways to cut the requested group into executed groups of one to kCostMaxConvs conv layers (a conv
    // stays with the pool after it) are then compared by the sum of their estimated pass times (found
    // from the last layer backwards), and the best one replaces the fixed rule's cuts when the model
    // puts it at least 3 % ahead; the margin keeps the model's error (about 10 % per group) from
    // trading a measured-good default for a predicted tie.
    auto estimate = [&](const GroupPlan& g) {
        if (g.st.on) return stationary_estimate_us(p, g, false, false) + stationary_estimate_us(p, g, true, g.first > 1);
        if (g.tfg.on) return tc_stationary_estimate_us(p, g, false, false) + tc_stationary_estimate_us(p, g, true, g.first > 1);
        double f[kCostTerms];
        pass_cost_terms(p, g, false, false, f);
        double t = pass_estimate_us(precision, false, f);
        pass_cost_terms(p, g, true, g.first > 1, f);
        return t + pass_estimate_us(precision, true, f);
    };
    p.groups.clear();
    for (int gi = 0; gi < n_groups; ++gi) {
        int start = groups[gi].first;
        const int first = start, last = groups[gi].last;
        std::vector<GroupPlan> cut;                        // the fixed rule's executed groups of this requested group
        while (start <= last) {
            GroupPlan g;
            double red = 1.0;
            int chosen = -1, last_rc = FTP_OK;
            int hi = std::min(last, start + kMaxOps - 1);
            if (!opts.strict_groups && opts.max_group_convs > 0) {
                int convs = 0, end = start - 1;
                bool alone_before = false;
                while (end + 1 <= hi) {
                    const bool is_conv = p.layers[end].kind == FTP_CONV;
                    if (is_conv && convs == opts.max_group_convs) break;
                    if (is_conv && convs > 0 && (alone_before || tc_stationary_conv(p, end, popts))) break;   // runs as a group of its own
                    if (is_conv) alone_before = tc_stationary_conv(p, end, popts);
                    if (is_conv && convs > 0 && p.layers[end - 1].kind == FTP_MAXPOOL) break;
                    if (is_conv) ++convs;
                    ++end;
                }
                hi = std::max(end, start);
            }
            if (opts.strict_groups) {
                if (hi != last) return FTP_ERR_GROUPS;
                int rc = make_group(p, lo, start, last, popts, g, &red);
                if (rc != FTP_OK) return rc;
                chosen = last;
            } else {
                // longest run of layers whose halo recomputation stays below the cap in both passes;
                // a conv is not separated from the pool after it unless nothing else works
                for (int pass = 0; pass < 3 && chosen < 0; ++pass)
                    for (int end = hi; end >= start; --end) {
                        const bool splits_pair = end < last && p.layers[end - 1].kind == FTP_CONV &&
                                                 p.layers[end].kind == FTP_MAXPOOL;
                        if (pass == 0 && splits_pair) continue;
                        int rc = make_group(p, lo, start, end, popts, g, &red);
                        last_rc = rc;
                        if (rc == FTP_OK && (pass == 2 || red * 100.0 <= opts.max_redundancy_pct)) { chosen = end; break; }
                    }
                if (chosen < 0) return last_rc == FTP_ERR_LAYERS ? FTP_ERR_LAYERS : FTP_ERR_WORKSPACE;
            }
            cut.push_back(g);
            start = chosen + 1;
        }
        if (opts.cost_model && !opts.strict_groups) {
            const double inf = 1e300;
            std::vector<double> best(last + 2, inf);
            std::vector<int> end_of(last + 2, -1);         // end_of[s]: last layer of the best executed group that starts at s
            best[last + 1] = 0;
            for (int s = last; s >= first; --s) {
                if (s > first && p.layers[s - 2].kind == FTP_CONV && p.layers[s - 1].kind == FTP_MAXPOOL) continue;
                int convs = 0;
                bool alone = false;
                for (int e = s; e <= std::min(last, s + kMaxOps - 1); ++e) {
                    if (p.layers[e - 1].kind == FTP_CONV && ++convs > kCostMaxConvs) break;
                    if (p.layers[e - 1].kind == FTP_CONV) alone = alone || tc_stationary_conv(p, e - 1, popts);
                    if (alone && convs > 1) break;             // such a conv is a group of its own
                    if (e < last && p.layers[e - 1].kind == FTP_CONV && p.layers[e].kind == FTP_MAXPOOL) continue;
                    if (best[e + 1] >= inf) continue;
                    GroupPlan g;
                    double red = 1.0;
                    if (make_group(p, lo, s, e, popts, g, &red) != FTP_OK || red * 100.0 > opts.max_redundancy_pct) continue;
                    const double cost = estimate(g) + best[e + 1];
                    if (cost < best[s]) { best[s] = cost; end_of[s] = e; }
                }
            }
            double fixed_cost = 0;
            for (const GroupPlan& g : cut) fixed_cost += estimate(g);
            if (best[first] < 0.97 * fixed_cost) {
                cut.clear();
                for (int s = first; s <= last; s = end_of[s] + 1) {
                    GroupPlan g;
                    if (end_of[s] < s || make_group(p, lo, s, end_of[s], popts, g, nullptr) != FTP_OK) return FTP_ERR_WORKSPACE;
                    cut.push_back(g);
                }
            }
        }
        for (const GroupPlan& g : cut) p.groups.push_back(g);
    }
    if (p.groups.size() > 64) return FTP_ERR_GROUPS;
    const int n_exec = (int)p.groups.size();

    // device tables
    p.tables.clear();
    auto push = [&](const std::vector<int>& v) { int o = (int)p.tables.size(); p.tables.insert(p.tables.end(), v.begin(), v.end()); return o; };
    for (GroupPlan& g : p.groups)
        for (PassPlan* pp : {&g.fwd, &g.bwd}) {
            pp->dev_yspan = push(pp->y.span);   pp->dev_xspan = push(pp->x.span);
            pp->dev_ycell = push(pp->y.cell);   pp->dev_xcell = push(pp->x.cell);
            pp->dev_yoff = push(pp->y.scratch_off); pp->dev_xoff = push(pp->x.scratch_off);
            pp->dev_ycover = push(pp->y.cover); pp->dev_xcover = push(pp->x.cover);
            pp->dev_ytile = push(pp->y.tile_begin); pp->dev_xtile = push(pp->x.tile_begin);
        }

    // workspace layout
    Workspace& ws = p.ws;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    ws.map_off.assign(n_layers + 1, 0);
    ws.arg_off.assign(n_layers + 1, 0);
    for (const GroupPlan& g : p.groups)
        for (int i = 0; i < g.n_ops; ++i) {
            const OpDesc& op = g.fwd_ops[i];
            const MapShape& s = p.maps[op.out_map - 1];
            if (tcp) {      // bf16 planes [n][C16/8][H][W][8]; arg-max bytes in the same arrangement
                const size_t c16 = (size_t)round_up(s.C, 16);
                ws.map_off[op.out_map - 1] = take((size_t)N * c16 * s.H * s.W * 2);
                if (op.kind == kOpConvPool) ws.arg_off[op.out_map - 1] = take((size_t)N * c16 * s.H * s.W);
                continue;
            }
            ws.map_off[op.out_map - 1] = take((size_t)N * s.C * s.H * s.W * 4);
            if (op.kind == kOpConvPool) ws.arg_off[op.out_map - 1] = take((size_t)N * s.C * s.H * s.W);
        }
    // Deltas at the inputs of the executed groups 1..: the backward pass of group gi reads the one at its output
    // (index gi + 1) and writes the one at its input (index gi), so two areas, taken in turn, hold them all.
    ws.dmap_off.assign(n_exec, 0);
    {
        size_t need[2] = {0, 0};
        for (int gi = 1; gi < n_exec; ++gi) {
            if (p.groups[gi].tfg.on && p.groups[gi - 1].tfg.on) continue;   // bf16 one-conv groups hand over dz planes instead
            const MapShape& s = p.maps[p.groups[gi].first - 1];
            const size_t bytes = tcp ? (size_t)N * round_up(s.C, 16) * s.H * s.W * 2     // bf16 planes
                                     : (size_t)N * s.C * s.H * s.W * 4;
            need[gi & 1] = std::max(need[gi & 1], bytes);
        }
        const size_t area[2] = {take(need[0]), take(need[1])};
        for (int gi = 1; gi < n_exec; ++gi) ws.dmap_off[gi] = area[gi & 1];
    }
    {
        const MapShape& s = p.maps[n_layers];
        ws.dy_off = take((size_t)N * s.C * s.H * s.W * 4);
        if (tcp) ws.y32_off = take((size_t)N * s.C * s.H * s.W * 4);
        size_t total = (size_t)N * s.C * s.H * s.W;
        p.loss_blocks = (int)std::min<size_t>(1024, (total + 1023) / 1024);
        ws.loss_off = take((size_t)p.loss_blocks * 4);
        ws.loss_val_off = take(4);
        ws.t_stage_bytes = align_up(total * 4, 256);                      // two staging slots each (ftp_prefetch_host)
        ws.x_stage_bytes = align_up((size_t)N * C * H * W * 4, 256);
        ws.t_stage_off = take(2 * ws.t_stage_bytes);
        ws.x_stage_off = take(2 * ws.x_stage_bytes);
    }
    // dz areas: fp32 one-conv groups take two equal areas in turn; bf16 one-conv groups use the first area for the
    // groups with an even index and the second for the odd ones (a group's input-delta kernel writes the dz planes
    // of the group below while it reads its own), each as large as its users need
    size_t scratch = 0, dz[2] = {0, 0};
    for (int gi = 0; gi < n_exec; ++gi) {
        const GroupPlan& g = p.groups[gi];
        scratch = std::max(scratch, g.bwd.scratch_floats);
        if (g.st.on && !g.st.thin)
            dz[0] = dz[1] = std::max(dz[0], (size_t)N * g.fwd_ops[0].cout * g.fwd_ops[0].in_H * g.fwd_ops[0].in_W * 4);
        if (g.tfg.on) dz[gi & 1] = std::max(dz[gi & 1], (size_t)N * g.fwd_ops[0].cout16 * g.fwd_ops[0].in_H * g.fwd_ops[0].in_W * 2);
        if (gi == 0 && g.col_cin16) dz[1] = std::max(dz[1], (size_t)N * g.col_cin16 * H * W * 2);   // delta of the unrolled input
    }
    ws.scratch_off = take(scratch * 4);
    if (!p.groups.empty() && p.groups[0].col_cin16) ws.col_off = take((size_t)N * p.groups[0].col_cin16 * H * W * 2);
    ws.dz_bytes = align_up(dz[0], 256);             // = offset of the second area
    ws.dz_off = take(ws.dz_bytes + align_up(dz[1], 256));
    ws.wf_off = take(p.wf_floats * (tcp ? 2 : 4));
    ws.wb_off = take(p.wb_floats * (tcp ? 2 : 4));
    ws.err_off = take(256);
    ws.partial_off = off;
    for (GroupPlan& g : p.groups) g.partial_off = take((size_t)g.sets() * g.param_floats * 4);
    ws.grad_off = take(p.param_floats * 4);
    ws.total = off;
    return FTP_OK;
}

int cost_terms(const ftp_plan& p, int pass, int group, int need_dx, double terms[kCostTerms], double* est_us)
{
    if (group < 0 || group >= (int)p.groups.size() || pass < 0 || pass > 1 || !terms) return FTP_ERR_ARG;
    pass_cost_terms(p, p.groups[group], pass == 1, need_dx != 0, terms);
    if (est_us) *est_us = p.groups[group].st.on  ? stationary_estimate_us(p, p.groups[group], pass == 1, need_dx != 0)
                        : p.groups[group].tfg.on ? tc_stationary_estimate_us(p, p.groups[group], pass == 1, need_dx != 0)
                                                 : pass_estimate_us(p.precision, pass == 1, terms);
    return FTP_OK;
}

int region(const ftp_plan& p, int pass, int group, int map_index, int ty, int tx, int out[4])
{
    if (!out || group < 0 || group >= (int)p.user_groups.size() || pass < 0 || pass > 2) return FTP_ERR_ARG;
    const ftp_group& g = p.user_groups[group];
    if (map_index < g.first || map_index > g.last + 1 || ty < 0 || ty >= p.grid_y || tx < 0 || tx >= p.grid_x)
        return FTP_ERR_ARG;
    const int m = map_index - g.first;      // 0 = group input
    Span sy, sx;
    if (pass == 0 || pass == 1) {
        const MapShape& om = p.maps[g.last];
        sy = equal_partition(0, om.H, p.grid_y)[ty];
        sx = equal_partition(0, om.W, p.grid_x)[tx];
        for (int i = g.last - g.first; i >= m; --i) {
            const ftp_layer& l = p.layers[g.first - 1 + i];
            sy = back_project(sy, l.k, l.stride, l.pad, p.maps[g.first - 1 + i].H);
            sx = back_project(sx, l.k, l.stride, l.pad, p.maps[g.first - 1 + i].W);
        }
    } else {
        const MapShape& in = p.maps[g.first - 1];
        sy = equal_partition(0, in.H, p.grid_y)[ty];
        sx = equal_partition(0, in.W, p.grid_x)[tx];
        for (int i = 0; i < m; ++i) {
            const ftp_layer& l = p.layers[g.first - 1 + i];
            sy = forward_project(sy, l.k, l.stride, l.pad, p.maps[g.first + i].H);
            sx = forward_project(sx, l.k, l.stride, l.pad, p.maps[g.first + i].W);
        }
    }
    out[0] = sx.a; out[1] = sy.a; out[2] = sx.b; out[3] = sy.b;
    return FTP_OK;
}

}  // namespace ftp
