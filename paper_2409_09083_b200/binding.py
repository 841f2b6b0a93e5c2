"""Thin ctypes binding of the C-ABI in include/ftp.h: argument marshalling only.

Every step of the path runs in the CUDA library.  If `libftp.so` has not been
built the import fails; there is no CPU fallback.  Tensors are torch CUDA
tensors (fp32, contiguous); torch is used for device memory and streams only.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.environ.get("FTP_LIBRARY") or os.path.join(_HERE, "libftp.so")   # FTP_LIBRARY: another build of the same library

if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2409_09083_b200.build` "
        "(there is no CPU fallback)")
_lib = ctypes.CDLL(_LIB_PATH)

FTP_CONV, FTP_MAXPOOL = 0, 1
FTP_FP32, FTP_BF16_FP32ACC = 0, 1


class ftp_layer(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("cin", ctypes.c_int), ("cout", ctypes.c_int),
                ("k", ctypes.c_int), ("stride", ctypes.c_int), ("pad", ctypes.c_int),
                ("leaky", ctypes.c_float)]


class ftp_group(ctypes.Structure):
    _fields_ = [("first", ctypes.c_int), ("last", ctypes.c_int)]


_vp, _i, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
_lib.ftp_plan_create.argtypes = [ctypes.POINTER(ftp_layer), _i, _i, _i, _i, _i, _i, _i,
                                 ctypes.POINTER(ftp_group), _i, _i, ctypes.POINTER(_vp)]
_lib.ftp_plan_create.restype = _i


class ftp_plan_opts(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_int), ("max_redundancy_pct", ctypes.c_int), ("max_subtile", ctypes.c_int),
                ("smem_bytes", ctypes.c_int), ("strict_groups", ctypes.c_int), ("tc_blocks_per_sm", ctypes.c_int), ("max_group_convs", ctypes.c_int), ("cost_model", ctypes.c_int),
                ("stationary", ctypes.c_int), ("tc_tma", ctypes.c_int)]


_lib.ftp_plan_create_opts.argtypes = [ctypes.POINTER(ftp_layer), _i, _i, _i, _i, _i, _i, _i,
                                      ctypes.POINTER(ftp_group), _i, _i, ctypes.POINTER(ftp_plan_opts),
                                      ctypes.POINTER(_vp)]
_lib.ftp_plan_create_opts.restype = _i
_lib.ftp_plan_exec_groups.argtypes = [_vp, ctypes.POINTER(_i), ctypes.POINTER(ftp_group), _i]
_lib.ftp_plan_exec_groups.restype = _i
_lib.ftp_plan_group_mode.argtypes = [_vp, _i, ctypes.POINTER(_i), ctypes.POINTER(_i)]
_lib.ftp_plan_group_mode.restype = _i
_lib.ftp_plan_destroy.argtypes = [_vp]
_lib.ftp_plan_destroy.restype = None
_lib.ftp_plan_region.argtypes = [_vp, _i, _i, _i, _i, _i, ctypes.POINTER(_i * 4)]
_lib.ftp_plan_region.restype = _i
_lib.ftp_plan_sizes.argtypes = [_vp, ctypes.POINTER(_sz), ctypes.POINTER(_sz), ctypes.POINTER(_sz),
                                ctypes.POINTER(ctypes.c_double)]
_lib.ftp_plan_sizes.restype = _i
_lib.ftp_plan_subtiles.argtypes = [_vp, _i, _i, ctypes.POINTER(_i), ctypes.POINTER(_i),
                                   ctypes.POINTER(_sz), ctypes.POINTER(_i)]
_lib.ftp_plan_subtiles.restype = _i
_lib.ftp_plan_delta_staging.argtypes = [_vp, _i, ctypes.POINTER(_i)]
_lib.ftp_plan_delta_staging.restype = _i
_lib.ftp_plan_cost.argtypes = [_vp, _i, _i, _i, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
_lib.ftp_plan_cost.restype = _i
_lib.ftp_forward.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp]
_lib.ftp_forward.restype = _i
_lib.ftp_backward.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.ftp_backward.restype = _i
_lib.ftp_step.argtypes = [_vp, _vp, _vp, _vp, _vp, ctypes.c_float, _vp, _vp, _vp, _vp]
_lib.ftp_step.restype = _i
_lib.ftp_step_host.argtypes = [_vp, _vp, _vp, _vp, ctypes.c_float, _vp, _vp, _vp, _vp]
_lib.ftp_step_host.restype = _i
_lib.ftp_prefetch_host.argtypes = [_vp, _vp, _vp, _vp, _vp]
_lib.ftp_prefetch_host.restype = _i
_lib.ftp_step_grad.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.ftp_step_grad.restype = _i
GROUP_READY_FN = ctypes.CFUNCTYPE(None, _vp, _i, ctypes.c_longlong, ctypes.c_longlong)
_lib.ftp_step_grad_groups.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, GROUP_READY_FN, _vp]
_lib.ftp_step_grad_groups.restype = _i
_lib.ftp_loss_mse.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.ftp_loss_mse.restype = _i
_lib.ftp_loss_mse_static.argtypes = [_vp, _vp, _vp, _vp, _sz, _vp]
_lib.ftp_loss_mse_static.restype = _i
_lib.ftp_sgd.argtypes = [_vp, _vp, _sz, ctypes.c_float, _vp]
_lib.ftp_sgd.restype = _i
_lib.ftp_fma_peak.argtypes = [_vp, _sz, ctypes.c_longlong, ctypes.POINTER(ctypes.c_double), _vp]
_lib.ftp_fma_peak.restype = _i


class ftp_launch_time(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("group", ctypes.c_int), ("ms", ctypes.c_float)]


_lib.ftp_plan_timing.argtypes = [_vp, _i]
_lib.ftp_plan_timing.restype = _i
_lib.ftp_plan_timing_read.argtypes = [_vp, ctypes.POINTER(_i), ctypes.POINTER(ftp_launch_time), _i]
_lib.ftp_plan_timing_read.restype = _i
_lib.ftp_plan_launch_count.argtypes = [_vp]
_lib.ftp_plan_launch_count.restype = ctypes.c_longlong
_lib.ftp_plan_check.argtypes = [_vp, _vp, _vp]
_lib.ftp_plan_check.restype = _i
_lib.ftp_plan_wait_probe.argtypes = [_vp, _vp, _i, _vp]
_lib.ftp_plan_wait_probe.restype = _i
_lib.ftp_strerror.argtypes = [_i]
_lib.ftp_strerror.restype = ctypes.c_char_p


class FtpError(RuntimeError):
    def __init__(self, code):
        self.code = code
        super().__init__(f"ftp error {code}: {_lib.ftp_strerror(code).decode()}")


def ftp_strerror(code: int) -> str:
    return _lib.ftp_strerror(code).decode()


def _check(rc):
    if rc != 0:
        raise FtpError(rc)


def _ptr(t, name, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise ValueError(f"{name} must not be None")
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous float32 CUDA tensor")
    return t.data_ptr()


def _sized(*specs):
    """Device pointers of tensors given as (tensor, name, element count[, allow_none]) after checking
    that each holds exactly that many elements: the kernels index by the plan's shapes, so a tensor
    of another size would be read or written out of bounds.  All sizes are checked before any
    pointer is taken."""
    for spec in specs:
        t, name, count = spec[:3]
        if t is not None and t.numel() != count:
            raise ValueError(f"{name} has {t.numel()} elements, the plan needs {count}")
    return [_ptr(spec[0], spec[1], len(spec) > 3 and spec[3]) for spec in specs]


class _Ws:
    """A workspace whose size has been checked; `.ptr` adds the device check, after the other arguments' sizes."""

    def __init__(self, plan, workspace):
        if workspace is None or not hasattr(workspace, "data_ptr"):
            raise ValueError("workspace must be a CUDA tensor of at least plan.workspace_bytes bytes")
        have = workspace.numel() * workspace.element_size()
        if have < plan.workspace_bytes:
            raise ValueError(f"workspace holds {have} bytes, the plan needs {plan.workspace_bytes}")
        self.t = workspace

    @property
    def ptr(self):
        if not self.t.is_cuda or not self.t.is_contiguous():
            raise ValueError("workspace must be a contiguous CUDA tensor")
        return self.t.data_ptr()


def _workspace(plan, workspace):
    return _Ws(plan, workspace)


def _host(*specs):
    """Host pointers of (tensor, name, element count) triples: sizes first, then layout."""
    for t, name, count in specs:
        if t is None:
            raise ValueError(f"{name} must not be None")
        if t.numel() != count:
            raise ValueError(f"{name} has {t.numel()} elements, the plan needs {count}")
    for t, name, _ in specs:
        if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous float32 CPU tensor")
    return [t.data_ptr() for t, _, _ in specs]


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _as_layers(layers):
    arr = (ftp_layer * len(layers))()
    for a, l in zip(arr, layers):
        conv = l.kind in ("conv", FTP_CONV)
        a.kind = FTP_CONV if conv else FTP_MAXPOOL
        a.cin, a.cout, a.k, a.stride, a.pad, a.leaky = l.cin, l.cout, l.k, l.stride, l.pad, l.leaky
    return arr


def _as_groups(groups):
    arr = (ftp_group * len(groups))()
    for a, g in zip(arr, groups):
        a.first, a.last = g
    return arr


class Plan:
    """Owner of an ftp_plan handle (ftp_plan_create / ftp_plan_destroy)."""

    def __init__(self, layers, N, C, H, W, grid, groups, precision=FTP_FP32, max_redundancy_pct=0, max_subtile=0,
                 smem_bytes=0, strict_groups=False, tc_blocks_per_sm=0, max_group_convs=0, cost_model=0, stationary=0, tc_tma=0):
        self._h = _vp()
        la, ga = _as_layers(layers), _as_groups(groups)
        opts = ftp_plan_opts(ctypes.sizeof(ftp_plan_opts), max_redundancy_pct, max_subtile, smem_bytes,
                             1 if strict_groups else 0, tc_blocks_per_sm, max_group_convs, int(cost_model), int(stationary), int(tc_tma))
        _check(_lib.ftp_plan_create_opts(la, len(layers), N, C, H, W, grid[0], grid[1], ga, len(groups),
                                         precision, ctypes.byref(opts), ctypes.byref(self._h)))
        self.layers, self.shape, self.grid, self.groups = list(layers), (N, C, H, W), tuple(grid), list(groups)
        pf, wb, of, red = _sz(), _sz(), _sz(), ctypes.c_double()
        _check(_lib.ftp_plan_sizes(self._h, ctypes.byref(pf), ctypes.byref(wb), ctypes.byref(of),
                                   ctypes.byref(red)))
        self.param_floats, self.workspace_bytes, self.out_floats = pf.value, wb.value, of.value
        self.in_floats = N * C * H * W
        self.redundancy = red.value

    def __del__(self):
        h = getattr(self, "_h", None)
        if h and _lib is not None:
            _lib.ftp_plan_destroy(h)
            self._h = None

    def exec_groups(self):
        """The grouping profile that is executed (a requested group may have been cut)."""
        n = _i()
        _check(_lib.ftp_plan_exec_groups(self._h, ctypes.byref(n), None, 0))
        arr = (ftp_group * n.value)()
        _check(_lib.ftp_plan_exec_groups(self._h, ctypes.byref(n), arr, n.value))
        return [(g.first, g.last) for g in arr]

    def group_mode(self, group):
        """(stationary, partial_sets) of executed group `group`: 1 if the weight-stationary kernels of the fp32 path run
        it, 2 if the banded tensor-core kernels of the bf16 path, 0 if it runs as fused sub-tile stacks; and how many
        partial gradient sets the cross-tile reduction sums for it."""
        st, sets = _i(), _i()
        _check(_lib.ftp_plan_group_mode(self._h, group, ctypes.byref(st), ctypes.byref(sets)))
        return st.value, sets.value

    def region(self, pass_, group, map_index, ty, tx):
        """(x1, y1, x2, y2), inclusive, of user tile (ty, tx) at map X_{map_index}."""
        out = (_i * 4)()
        _check(_lib.ftp_plan_region(self._h, pass_, group, map_index, ty, tx, ctypes.byref(out)))
        return tuple(out)

    def subtiles(self, pass_, group):
        r, c, s, b = _i(), _i(), _sz(), _i()
        _check(_lib.ftp_plan_subtiles(self._h, pass_, group, ctypes.byref(r), ctypes.byref(c),
                                      ctypes.byref(s), ctypes.byref(b)))
        return dict(rows=r.value, cols=c.value, smem_bytes=s.value, blocks=b.value)

    def delta_staging(self, group):
        """Channels of the backward pass's delta staging area of an executed group (fp32 path; 0 = none)."""
        ch = _i()
        _check(_lib.ftp_plan_delta_staging(self._h, group, ctypes.byref(ch)))
        return ch.value

    def cost(self, pass_, group, need_dx=True):
        """(terms, estimate in microseconds) of the planner's time model for one pass of an executed group."""
        terms = (ctypes.c_double * 8)()
        est = ctypes.c_double()
        _check(_lib.ftp_plan_cost(self._h, pass_, group, 1 if need_dx else 0, terms, ctypes.byref(est)))
        return list(terms), est.value

    def launch_count(self):
        return int(_lib.ftp_plan_launch_count(self._h))

    def timing(self, enable=True):
        _check(_lib.ftp_plan_timing(self._h, 1 if enable else 0))

    def timing_read(self):
        """[(kind, group, ms)] of the launches since the last read; synchronise the stream first."""
        cap = 512
        arr = (ftp_launch_time * cap)()
        n = _i()
        _check(_lib.ftp_plan_timing_read(self._h, ctypes.byref(n), arr, cap))
        return [(arr[i].kind, arr[i].group, arr[i].ms) for i in range(min(n.value, cap))]

    def check(self, workspace, stream=None):
        """Synchronise and raise FtpError(FTP_ERR_TIMEOUT) if a device-side wait of the bf16 path ran out."""
        _check(_lib.ftp_plan_check(self._h, _workspace(self, workspace).ptr, _stream(stream)))

    def wait_probe(self, workspace, limit_us=2000, stream=None):
        """Launches the kernel whose bounded wait runs out on purpose (see ftp_plan_wait_probe in ftp.h)."""
        _check(_lib.ftp_plan_wait_probe(self._h, _workspace(self, workspace).ptr, int(limit_us), _stream(stream)))

    def new_workspace(self, device="cuda"):
        return torch.empty(self.workspace_bytes, dtype=torch.uint8, device=device)


def ftp_plan(layers, N, C, H, W, tile_grid, groups, precision=FTP_FP32, **opts) -> Plan:
    return Plan(layers, N, C, H, W, tile_grid, groups, precision, **opts)


def ftp_forward(plan, x, params, y, workspace, stream=None):
    ws = _workspace(plan, workspace)
    px, pp, py = _sized((x, "x", plan.in_floats), (params, "params", plan.param_floats), (y, "y", plan.out_floats, True))
    _check(_lib.ftp_forward(plan._h, px, pp, py, ws.ptr, _stream(stream)))


def ftp_backward(plan, x, dy, params, dx, dparams, workspace, stream=None):
    ws = _workspace(plan, workspace)
    px, pdy, pp, pdx, pg = _sized((x, "x", plan.in_floats), (dy, "dy", plan.out_floats),
                                  (params, "params", plan.param_floats), (dx, "dx", plan.in_floats, True),
                                  (dparams, "dparams", plan.param_floats))
    _check(_lib.ftp_backward(plan._h, px, pdy, pp, pdx, pg, ws.ptr, _stream(stream)))


def ftp_step(plan, x, params, lr, workspace, dy=None, target=None, loss_out=None, dx=None, stream=None):
    ws = _workspace(plan, workspace)
    px, pdy, pt, pp, pl, pdx = _sized((x, "x", plan.in_floats), (dy, "dy", plan.out_floats, True),
                                      (target, "target", plan.out_floats, True), (params, "params", plan.param_floats),
                                      (loss_out, "loss_out", 1, True), (dx, "dx", plan.in_floats, True))
    _check(_lib.ftp_step(plan._h, px, pdy, pt, pp, float(lr), pl, pdx, ws.ptr, _stream(stream)))


def ftp_step_grad(plan, x, params, dparams, workspace, dy=None, target=None, loss_out=None, dx=None, stream=None):
    ws = _workspace(plan, workspace)
    px, pdy, pt, pp, pg, pl, pdx = _sized((x, "x", plan.in_floats), (dy, "dy", plan.out_floats, True),
                                          (target, "target", plan.out_floats, True),
                                          (params, "params", plan.param_floats), (dparams, "dparams", plan.param_floats),
                                          (loss_out, "loss_out", 1, True), (dx, "dx", plan.in_floats, True))
    _check(_lib.ftp_step_grad(plan._h, px, pdy, pt, pp, pg, pl, pdx, ws.ptr, _stream(stream)))


def ftp_step_grad_groups(plan, x, params, dparams, workspace, ready, dy=None, target=None, loss_out=None, dx=None, stream=None):
    """ftp_step_grad that calls ready(group, param_begin, param_floats) on the host as soon as the launches that
    complete an executed group's slice of dparams are queued on the stream (groups finish in reverse order)."""
    ws = _workspace(plan, workspace)
    px, pdy, pt, pp, pg, pl, pdx = _sized((x, "x", plan.in_floats), (dy, "dy", plan.out_floats, True),
                                          (target, "target", plan.out_floats, True),
                                          (params, "params", plan.param_floats), (dparams, "dparams", plan.param_floats),
                                          (loss_out, "loss_out", 1, True), (dx, "dx", plan.in_floats, True))
    errors = []

    def trampoline(_user, group, begin, count):
        try:
            ready(int(group), int(begin), int(count))
        except BaseException as e:            # noqa: BLE001 - must not unwind through the C frames
            errors.append(e)
    cb = GROUP_READY_FN(trampoline)
    rc = _lib.ftp_step_grad_groups(plan._h, px, pdy, pt, pp, pg, pl, pdx, ws.ptr, _stream(stream), cb, None)
    if errors:
        raise errors[0]
    _check(rc)


def ftp_loss_mse(plan, y, target, dy, loss_out, workspace, stream=None):
    ws = _workspace(plan, workspace)
    py, pt, pdy, pl = _sized((y, "y", plan.out_floats), (target, "target", plan.out_floats),
                             (dy, "dy", plan.out_floats, True), (loss_out, "loss_out", 1, True))
    _check(_lib.ftp_loss_mse(plan._h, py, pt, pdy, pl, ws.ptr, _stream(stream)))


def ftp_loss_mse_static(y, target, dy, loss_out, stream=None):
    """MSE loss and delta without a plan, a workspace or any device allocation (see ftp.h)."""
    if y is None or target is None:
        raise ValueError("y and target must not be None")
    py, pt, pdy, pl = _sized((y, "y", y.numel()), (target, "target", y.numel()), (dy, "dy", y.numel(), True),
                             (loss_out, "loss_out", 1, True))
    _check(_lib.ftp_loss_mse_static(py, pt, pdy, pl, y.numel(), _stream(stream)))


def ftp_sgd(params, grad, lr, stream=None):
    if params is None:
        raise ValueError("params must not be None")
    pp, pg = _sized((params, "params", params.numel()), (grad, "grad", params.numel()))
    _check(_lib.ftp_sgd(pp, pg, params.numel(), float(lr), _stream(stream)))


def ftp_fma_peak(out, iters, stream=None):
    """Launches the register-only fp32 FMA loop (see ftp.h); returns the floating-point operations it performs."""
    flops = ctypes.c_double()
    (po,) = _sized((out, "out", out.numel()))
    _check(_lib.ftp_fma_peak(po, out.numel(), int(iters), ctypes.byref(flops), _stream(stream)))
    return flops.value


def ftp_prefetch_host(plan, x_host, target_host, workspace, copy_stream=None):
    """Starts copying the NEXT batch (pinned float32 CPU tensors) while the current step runs; the
    ftp_step_host call given the same two tensors then waits for these copies instead of copying.
    copy_stream=None selects the plan's own side stream (the NULL of the C-ABI), whatever stream is
    current, so that the copies never queue behind the step they are meant to overlap."""
    px, pt = _host((x_host, "x_host", plan.in_floats), (target_host, "target_host", plan.out_floats))
    _check(_lib.ftp_prefetch_host(plan._h, px, pt, _workspace(plan, workspace).ptr,
                                  None if copy_stream is None else _stream(copy_stream)))


def ftp_step_host(plan, x_host, target_host, params, lr, loss_host, workspace, dx=None, stream=None):
    """x_host, target_host, loss_host: float32 CPU tensors (pinned memory recommended)."""
    px, pt, pl = _host((x_host, "x_host", plan.in_floats), (target_host, "target_host", plan.out_floats),
                       (loss_host, "loss_host", 1))
    ws = _workspace(plan, workspace)
    pp, pdx = _sized((params, "params", plan.param_floats), (dx, "dx", plan.in_floats, True))
    _check(_lib.ftp_step_host(plan._h, px, pt, pp, float(lr), pl, pdx, ws.ptr, _stream(stream)))
