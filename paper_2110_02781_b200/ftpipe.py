"""ctypes binding of libftpipe.so: argument marshalling only, one function per C entry point,
same names.  Device buffers are torch tensors (torch provides device memory and streams);
every step of the path runs inside the library's kernels.

There is no fallback: importing this module without the built library raises.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("FTPIPE_LIB") or os.path.join(_HERE, "libftpipe.so")       # FTPIPE_LIB: another build of the library (measurement variants)
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2110_02781_b200.build`")
lib = C.CDLL(LIB_PATH)

OK = 0
STATUS = {0: "FTP_OK", 1: "FTP_EINVAL", 2: "FTP_ERANGE", 3: "FTP_ENOMEM", 4: "FTP_ECUDA", 5: "FTP_ESTATE",
          6: "FTP_ETIMEOUT", 7: "FTP_EUNSUPPORTED"}
T_WEIGHTS, T_GRADS, T_MOMENTUM, T_STATE = 0, 1, 2, 3
FP32, BF16 = 0, 1


class LayerDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("unit", "kind", "cin", "cout", "k", "stride", "pad", "act", "has_bias",
                                          "residual_src")]


class ModelCfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "in_c", "in_h", "in_w", "n_classes", "precision", "max_stages")] + \
               [(n, C.c_float) for n in ("lr", "momentum", "weight_decay", "bn_eps", "bn_momentum")]


class TraceRec(C.Structure):
    _fields_ = [("kernel", C.c_int32), ("unit", C.c_int32), ("op", C.c_int32), ("backward", C.c_int32),
                ("ms", C.c_float), ("bytes", C.c_double), ("flops", C.c_double)]


class TrainState(C.Structure):
    _fields_ = [("committed_forward_id", C.c_int64), ("committed_backward_id", C.c_int64), ("status", C.c_int32),
                ("learning_rate", C.c_float), ("epoch_number", C.c_int64), ("batch_number", C.c_int64)]


PROBE_NORMAL, PROBE_RESTARTED, PROBE_SILENT = 0, 1, 2
ACTION_RESTART_BATCH, ACTION_RESEND_STATE, ACTION_REDISTRIBUTE = 0, 1, 2


class FtpError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"{STATUS.get(status, status)}: {text}")
        self.status = status


_vp, _i32, _i64, _sz, _f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t, C.c_float
_P = C.POINTER
_SIGS = {
    "ftp_workspace_bytes": [_P(LayerDesc), _i32, _P(ModelCfg), _P(_sz), _P(_sz)],
    "ftp_build_model": [_P(LayerDesc), _i32, _P(ModelCfg), _vp, _sz, _vp, _sz, _P(_vp)],
    "ftp_num_units": [_vp, _P(_i32)],
    "ftp_unit_param_span": [_vp, _i32, _P(_i64), _P(_i64)],
    "ftp_unit_state_span": [_vp, _i32, _P(_i64), _P(_i64)],
    "ftp_unit_output_shape": [_vp, _i32, _P(_i32), _P(_i64)],
    "ftp_set_tensor": [_vp, _i32, _i32, _vp, _i64, _i32, _vp],
    "ftp_get_tensor": [_vp, _i32, _i32, _vp, _i64, _i32, _vp],
    "ftp_run_stage_forward": [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp],
    "ftp_run_stage_backward": [_vp, _i32, _i32, _vp, _vp, _vp],
    "ftp_get_logits": [_vp, _vp, _i32, _vp],
    "ftp_sgd_step": [_vp, _i32, _i32, _f32, _vp, _vp, _vp],
    "ftp_train_step": [_vp, _vp, _vp, _i32, _f32, _P(_f32), _vp],
    "ftp_profile_layers": [_vp, _i32, _vp, _vp, _P(C.c_double), _P(C.c_double), _P(_i64), _vp],
    "ftp_estimate_capacity": [_P(C.c_double), _i32, _P(_i32), _i32, _P(C.c_double), _P(C.c_double)],
    "ftp_choose_partition": [_P(C.c_double), _i32, _P(C.c_double), _i32, _P(C.c_double), _P(C.c_double), _P(_i32),
                             _P(C.c_double)],
    "ftp_redistribution_plan": [_P(_i32), _i32, _P(_i32), _i32, _i32, _i32, _i32, _P(_i32), _P(_i32)],
    "ftp_stage_timing_enable": [_vp, _i32],
    "ftp_stage_times": [_vp, _P(C.c_double), _P(_i32)],
    "ftp_recovery_plan": [_P(_i32), _i32, _P(_i32), _i32, _P(_i32), _i32, _P(_i32), _P(_i32)],
    "ftp_recover": [_vp, _vp, _i32, _vp, _sz, _P(_i32), _i32, _P(_i32), _vp],
    "ftp_set_partition": [_vp, _P(_i32), _i32, _P(_i32), _vp],
    "ftp_get_partition": [_vp, _P(_i32), _P(_i32)],
    "ftp_snapshot_weights": [_vp, _i32, _vp, _sz, _i32, _P(_sz), _vp],
    "ftp_state_init": [_P(TrainState), _f32, _i64, _i64],
    "ftp_state_forward_done": [_P(TrainState), _i64],
    "ftp_state_backward_done": [_P(TrainState), _i64],
    "ftp_state_timer_expired": [_P(TrainState), _i64, _P(_i32)],
    "ftp_state_may_forward": [_P(TrainState), _i64, _P(_i32)],
    "ftp_state_reset": [_P(TrainState), _i64, _P(_i64)],
    "ftp_classify_probe": [_P(_i32), _i32, _P(_i32), _P(_i32), _P(_i32), _P(_i32)],
    "ftp_async_stage_order": [_i32, _i32, _i32, _P(_i32), _P(_i32)],
    "ftp_async_version_trace": [_i32, _i32, _i32, _i32, _P(_i64), _P(_i64), _P(_i32)],
    "ftp_sync_units": [_vp, _vp, _i32, _i32, _i32, _vp],
    "ftp_sgd_step_from": [_vp, _vp, _i32, _i32, _f32, _vp],
    "ftp_aggregate_weights": [_vp, _P(_vp), _i32, _i32, _i32, _vp],
    "ftp_measure_bandwidth": [_vp, _vp, _sz, _i32, _P(C.c_double), _P(C.c_double), _vp],
    "ftp_check_guards": [_vp, _P(_i32), _P(_i64), _vp],
    "ftp_check_device_status": [_vp, _vp],
    "ftp_debug_set_device_status": [_vp, _i32, _vp],
    "ftp_trace_enable": [_vp, _i32],
    "ftp_trace_read": [_vp, _P(TraceRec), _i32, _P(_i32)],
    "ftp_launch_count": [_vp, _P(_i64)],
    "ftp_conv_wgrad_static": [_vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32, _i32, _i32, _i32, _vp],
}
for _name, _args in _SIGS.items():
    _f = getattr(lib, _name)
    _f.argtypes, _f.restype = _args, C.c_int
lib.ftp_destroy_model.argtypes, lib.ftp_destroy_model.restype = [_vp], None
lib.ftp_last_error.argtypes, lib.ftp_last_error.restype = [], C.c_char_p
lib.ftp_kernel_name.argtypes, lib.ftp_kernel_name.restype = [_i32], C.c_char_p
lib.ftp_is_repartition_iter.argtypes, lib.ftp_is_repartition_iter.restype = [_i64, _i64, _i64], _i32
lib.ftp_is_replication_iter.argtypes, lib.ftp_is_replication_iter.restype = [_i64, _i64], _i32


def _check(status):
    if status != OK:
        raise FtpError(status, lib.ftp_last_error().decode())


def _ptr(t):
    """Address of a torch tensor / numpy array / raw int, or NULL."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _dbl(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(_P(C.c_double))


def _i32arr(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(_P(_i32))


def layer_array(layers):
    arr = (LayerDesc * len(layers))()
    for i, l in enumerate(layers):
        arr[i] = LayerDesc(*[int(v) for v in l])
    return arr


def model_cfg(cfg):
    return ModelCfg(cfg["batch"], cfg["in_c"], cfg["in_h"], cfg["in_w"], cfg["n_classes"], cfg["precision"],
                    cfg["max_stages"], cfg["lr"], cfg["momentum"], cfg["weight_decay"], cfg["bn_eps"], cfg["bn_momentum"])


# ---- pure host functions (usable without a GPU) ------------------------------------------------
def ftp_estimate_capacity(layer_times, points, stage_times):
    lt, plt = _dbl(layer_times)
    pts, ppts = _i32arr(points)
    stt, pst = _dbl(stage_times)
    out = np.zeros(len(pts) - 1, np.float64)
    _check(lib.ftp_estimate_capacity(plt, len(lt), ppts, len(pts) - 1, pst, out.ctypes.data_as(_P(C.c_double))))
    return out.tolist()


def ftp_choose_partition(layer_times, capacities, out_bytes=None, bandwidth=None):
    lt, plt = _dbl(layer_times)
    cp, pcp = _dbl(capacities)
    ob = bw = pob = pbw = None
    if out_bytes is not None:
        ob, pob = _dbl(out_bytes)
    if bandwidth is not None:
        bw, pbw = _dbl(bandwidth)
    pts = np.zeros(len(cp) + 1, np.int32)
    bott = C.c_double()
    _check(lib.ftp_choose_partition(plt, len(lt), pcp, len(cp), pob, pbw, pts.ctypes.data_as(_P(_i32)), C.byref(bott)))
    return pts.tolist(), bott.value


def ftp_redistribution_plan(p_new, p_cur, i_cur, i_new, i_fail=-1):
    pn, ppn = _i32arr(p_new)
    pc, ppc = _i32arr(p_cur)
    if not (0 <= i_new < len(pn) - 1):
        raise FtpError(2, "i_new out of range")
    owners = np.full(max(int(pn[i_new + 1] - pn[i_new]), 1), -7, np.int32)
    nloc = _i32()
    _check(lib.ftp_redistribution_plan(ppn, len(pn) - 1, ppc, len(pc) - 1, i_fail, i_cur, i_new,
                                       owners.ctypes.data_as(_P(_i32)), C.byref(nloc)))
    return owners[:int(pn[i_new + 1] - pn[i_new])].tolist(), nloc.value


SRC_LOCAL, SRC_STAGE, SRC_REPLICA, SRC_CENTRAL = 0, 1, 2, 3


class FailedStage(C.Structure):
    _fields_ = [("stage", _i32), ("replica_is_host", _i32), ("replica", _vp), ("replica_bytes", _sz)]


def ftp_recovery_plan(p_cur, failed, p_new):
    """Per unit: (kind, index) as ftp_recovery_plan in include/ftpipe.h defines them."""
    pc, ppc = _i32arr(p_cur)
    pn, ppn = _i32arr(p_new)
    fl, pfl = _i32arr(failed)
    L = int(pc[-1])
    kind, index = np.full(max(L, 1), -7, np.int32), np.full(max(L, 1), -7, np.int32)
    _check(lib.ftp_recovery_plan(ppc, len(pc) - 1, pfl, len(fl), ppn, len(pn) - 1, kind.ctypes.data_as(_P(_i32)),
                                 index.ctypes.data_as(_P(_i32))))
    return kind[:L].tolist(), index[:L].tolist()


def ftp_state_init(learning_rate, epoch_number, batch_number):
    st = TrainState()
    _check(lib.ftp_state_init(C.byref(st), learning_rate, epoch_number, batch_number))
    return st


def ftp_state_forward_done(st, batch_id):
    _check(lib.ftp_state_forward_done(C.byref(st), batch_id))


def ftp_state_backward_done(st, batch_id):
    _check(lib.ftp_state_backward_done(C.byref(st), batch_id))


def ftp_state_timer_expired(st, batch_id):
    t = _i32()
    _check(lib.ftp_state_timer_expired(C.byref(st), batch_id, C.byref(t)))
    return bool(t.value)


def ftp_state_may_forward(st, batch_id):
    a = _i32()
    _check(lib.ftp_state_may_forward(C.byref(st), batch_id, C.byref(a)))
    return bool(a.value)


def ftp_state_reset(st, batch_id):
    r = _i64()
    _check(lib.ftp_state_reset(C.byref(st), batch_id, C.byref(r)))
    return r.value


def ftp_classify_probe(responses):
    n = len(responses)
    r = (_i32 * n)(*responses)
    failed = (_i32 * n)()
    action, nf, rw = _i32(), _i32(), _i32()
    _check(lib.ftp_classify_probe(r, n, C.byref(action), failed, C.byref(nf), C.byref(rw)))
    return action.value, list(failed[:nf.value]), (rw.value if rw.value >= 0 else None)


def ftp_is_repartition_iter(it, first=10, period=100):
    return bool(lib.ftp_is_repartition_iter(it, first, period))


def ftp_is_replication_iter(it, period):
    return bool(lib.ftp_is_replication_iter(it, period))


SYNC_WEIGHTS, SYNC_MOMENTUM, SYNC_STATE = 1, 2, 4


def ftp_async_stage_order(n_stages, stage, n_batches):
    isb, bat = (_i32 * (2 * n_batches + 1))(), (_i32 * (2 * n_batches + 1))()
    _check(lib.ftp_async_stage_order(n_stages, stage, n_batches, isb, bat))
    return [("B" if isb[e] else "F", bat[e]) for e in range(2 * n_batches)]


def ftp_async_version_trace(n_stages, stage, n_batches, k=1):
    fv, av, ag = (_i64 * max(n_batches, 1))(), (_i64 * max(n_batches, 1))(), (_i32 * max(n_batches, 1))()
    _check(lib.ftp_async_version_trace(n_stages, stage, n_batches, k, fv, av, ag))
    return list(fv[:n_batches]), list(av[:n_batches]), [b for b in range(n_batches) if ag[b]]


def ftp_sync_units(dst, src, a, b, what, stream=None):
    _check(lib.ftp_sync_units(dst.h, src.h, a, b, what, _stream(stream)))


def ftp_sgd_step_from(dst, grads, a, b, lr, stream=None):
    _check(lib.ftp_sgd_step_from(dst.h, grads.h, a, b, lr, _stream(stream)))


def ftp_aggregate_weights(dst, srcs, a, b, stream=None):
    arr = (_vp * len(srcs))(*[m.h for m in srcs])
    _check(lib.ftp_aggregate_weights(dst.h, arr, len(srcs), a, b, _stream(stream)))


def ftp_workspace_bytes(layers, cfg):
    d, p = _sz(), _sz()
    _check(lib.ftp_workspace_bytes(layer_array(layers), len(layers), C.byref(model_cfg(cfg)), C.byref(d), C.byref(p)))
    return d.value, p.value


def ftp_conv_wgrad_static(x, dy, dw, k, stride, pad, stream=None):
    """Weight gradient of a dense k x k convolution without any workspace argument, for callers that
    may not allocate device memory: x (n, h, w, cin), dy (n, ho, wo, cout) and dw (k, k, cin, cout)
    are float32 CUDA tensors the caller already owns.  See include/ftpipe.h for the limits."""
    import torch
    def bad(why):
        raise FtpError(1, "conv_wgrad_static: " + why)
    for name, t in (("x", x), ("dy", dy), ("dw", dw)):
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
            bad(f"{name} must be a contiguous float32 CUDA tensor")
        if t.device != x.device:
            bad("x, dy and dw must live on one device")
    if x.device.index != torch.cuda.current_device():
        bad("the tensors' device must be the current device")
    if x.dim() != 4 or dy.dim() != 4 or k < 1 or stride < 1 or pad < 0:
        bad("x and dy must be 4-D (n, h, w, c); k, stride >= 1, pad >= 0")
    n, h, w, cin = x.shape
    if h + 2 * pad < k or w + 2 * pad < k:
        bad("kernel larger than the padded input")
    ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
    if tuple(dy.shape[:3]) != (n, ho, wo):
        bad(f"dy must be ({n}, {ho}, {wo}, cout), got {tuple(dy.shape)}")
    if tuple(dw.shape) != (k, k, cin, dy.shape[3]):
        bad(f"dw must be ({k}, {k}, {cin}, {dy.shape[3]}), got {tuple(dw.shape)}")
    _check(lib.ftp_conv_wgrad_static(_ptr(x), _ptr(dy), _ptr(dw), n, h, w, cin, dy.shape[3], k, stride, pad,
                                     _stream(stream)))


def ftp_kernel_name(k):
    return lib.ftp_kernel_name(k).decode()


# ---- the model -----------------------------------------------------------------------------------
class Model:
    """Owns the workspaces (torch device memory + pinned host memory) and the ftp_model handle.
    Methods are the C entry points with the handle bound."""

    def __init__(self, layers, cfg, device="cuda:0"):
        import torch
        self.torch = torch
        self.layers, self.cfg = list(layers), dict(cfg)
        self.device = torch.device(device)
        dev_bytes, pin_bytes = ftp_workspace_bytes(layers, cfg)
        self.dev_ws = torch.empty(dev_bytes + 256, dtype=torch.uint8, device=self.device)
        self.pin_ws = torch.empty(max(pin_bytes, 256), dtype=torch.uint8).pin_memory()
        base = (self.dev_ws.data_ptr() + 255) // 256 * 256
        h = _vp()
        with torch.cuda.device(self.device):
            _check(lib.ftp_build_model(layer_array(layers), len(layers), C.byref(model_cfg(cfg)), base, dev_bytes,
                                       self.pin_ws.data_ptr(), self.pin_ws.numel(), C.byref(h)))
        self.h = h
        n = _i32()
        _check(lib.ftp_num_units(self.h, C.byref(n)))
        self.L = n.value
        self.act_dtype = torch.bfloat16 if cfg["precision"] == BF16 else torch.float32

    def close(self):
        if getattr(self, "h", None) and lib is not None:        # lib is None while the interpreter shuts down
            lib.ftp_destroy_model(self.h)
            self.h = None

    __del__ = close

    def ftp_unit_param_span(self, unit):
        o, c = _i64(), _i64()
        _check(lib.ftp_unit_param_span(self.h, unit, C.byref(o), C.byref(c)))
        return o.value, c.value

    def ftp_unit_state_span(self, unit):
        o, c = _i64(), _i64()
        _check(lib.ftp_unit_state_span(self.h, unit, C.byref(o), C.byref(c)))
        return o.value, c.value

    def ftp_unit_output_shape(self, unit):
        shp = (_i32 * 4)()
        b = _i64()
        _check(lib.ftp_unit_output_shape(self.h, unit, shp, C.byref(b)))
        return tuple(shp), b.value

    def ftp_set_tensor(self, which, unit, src, stream=None):
        """src: float32 numpy array (host) or torch CUDA tensor (device)."""
        dev = not isinstance(src, np.ndarray)
        if not dev:
            src = np.ascontiguousarray(src, dtype=np.float32)
        n = src.size if not dev else src.numel()
        _check(lib.ftp_set_tensor(self.h, which, unit, _ptr(src), n, int(dev), _stream(stream)))

    def ftp_get_tensor(self, which, unit, stream=None):
        """Returns a float32 numpy array (host copy)."""
        n = self.ftp_unit_state_span(unit)[1] if which == T_STATE else self.ftp_unit_param_span(unit)[1]
        out = np.empty(n, np.float32)
        _check(lib.ftp_get_tensor(self.h, which, unit, _ptr(out), n, 0, _stream(stream)))
        return out

    def ftp_run_stage_forward(self, a, b, act_in, act_out=None, labels=None, loss_out=None, stream=None):
        _check(lib.ftp_run_stage_forward(self.h, a, b, _ptr(act_in), _ptr(act_out), _ptr(labels), _ptr(loss_out),
                                         _stream(stream)))

    def ftp_run_stage_backward(self, a, b, grad_out=None, grad_in=None, stream=None):
        _check(lib.ftp_run_stage_backward(self.h, a, b, _ptr(grad_out), _ptr(grad_in), _stream(stream)))

    def ftp_get_logits(self, stream=None):
        out = np.empty((self.cfg["batch"], self.cfg["n_classes"]), np.float32)
        _check(lib.ftp_get_logits(self.h, _ptr(out), 0, _stream(stream)))
        return out

    def ftp_sgd_step(self, a, b, lr, snap_dev=None, snap_host=None, stream=None):
        _check(lib.ftp_sgd_step(self.h, a, b, lr, _ptr(snap_dev), _ptr(snap_host), _stream(stream)))

    def ftp_train_step(self, x, labels, lr, inputs_on_host=False, want_loss=True, stream=None, loss_pinned=None):
        """loss_pinned: a pinned float32 host tensor of one element that receives the loss instead of the return value --
        the form to use while the step is captured into a CUDA graph (the copy becomes a node of the graph)."""
        if loss_pinned is not None:
            if loss_pinned.is_cuda or not loss_pinned.is_pinned() or loss_pinned.numel() < 1 or loss_pinned.element_size() != 4:
                raise ValueError("loss_pinned must be a pinned float32 host tensor")
            _check(lib.ftp_train_step(self.h, _ptr(x), _ptr(labels), int(inputs_on_host), lr,
                                      C.cast(loss_pinned.data_ptr(), _P(_f32)), _stream(stream)))
            return None
        loss = _f32()
        _check(lib.ftp_train_step(self.h, _ptr(x), _ptr(labels), int(inputs_on_host), lr,
                                  C.byref(loss) if want_loss else None, _stream(stream)))
        return loss.value if want_loss else None

    def ftp_stage_timing_enable(self, on):
        _check(lib.ftp_stage_timing_enable(self.h, int(on)))

    def ftp_stage_times(self):
        """Forward + backward device seconds of every stage in the last timed ftp_train_step."""
        t = (C.c_double * self.cfg["max_stages"])()
        n = _i32()
        _check(lib.ftp_stage_times(self.h, t, C.byref(n)))
        return list(t[:n.value])

    def ftp_profile_layers(self, reps, sample_in, labels, stream=None):
        f, b = np.zeros(self.L), np.zeros(self.L)
        ob = np.zeros(self.L, np.int64)
        _check(lib.ftp_profile_layers(self.h, reps, _ptr(sample_in), _ptr(labels), f.ctypes.data_as(_P(C.c_double)),
                                      b.ctypes.data_as(_P(C.c_double)), ob.ctypes.data_as(_P(_i64)), _stream(stream)))
        return f, b, ob

    def ftp_set_partition(self, points, stream=None):
        pts, pp = _i32arr(points)
        moved = _i32()
        _check(lib.ftp_set_partition(self.h, pp, len(pts) - 1, C.byref(moved), _stream(stream)))
        return moved.value

    def ftp_recover(self, failed, p_new, central=None, stream=None):
        """failed: {stage: chain replica tensor (device, or host for the last stage) or None}; central: the global
        replica (host tensor, all units in canonical order) or None.  Returns (from stages, from replicas, from central)."""
        recs = (FailedStage * max(len(failed), 1))()
        for k, (stage, rep) in enumerate(sorted(failed.items())):
            recs[k].stage = stage
            recs[k].replica_is_host = int(rep is not None and not rep.is_cuda)
            recs[k].replica = _ptr(rep)
            recs[k].replica_bytes = 0 if rep is None else rep.numel() * rep.element_size()
        pts, pp = _i32arr(p_new)
        counts = (_i32 * 3)()
        _check(lib.ftp_recover(self.h, recs, len(failed), _ptr(central), 0 if central is None else central.numel() * central.element_size(),
                               pp, len(pts) - 1, counts, _stream(stream)))
        return tuple(counts)

    def ftp_get_partition(self):
        pts = (_i32 * (self.cfg["max_stages"] + 1))()
        n = _i32()
        _check(lib.ftp_get_partition(self.h, pts, C.byref(n)))
        return list(pts[:n.value + 1])

    def ftp_snapshot_weights(self, stage, dst, stream=None):
        """dst: torch tensor, device or pinned host (float32)."""
        w = _sz()
        _check(lib.ftp_snapshot_weights(self.h, stage, _ptr(dst), dst.numel() * dst.element_size(),
                                        int(not dst.is_cuda), C.byref(w), _stream(stream)))
        return w.value

    def ftp_measure_bandwidth(self, pinned_host=None, nbytes=64 << 20, reps=5, stream=None):
        """(device-to-device, device-to-pinned-host) copy bandwidth in bytes per second."""
        a, b = C.c_double(), C.c_double()
        _check(lib.ftp_measure_bandwidth(self.h, _ptr(pinned_host), nbytes, reps, C.byref(a), C.byref(b), _stream(stream)))
        return a.value, b.value

    def ftp_check_guards(self, stream=None):
        """Number of guard zones checked; raises FtpError (with .bad_offset) if one was overwritten."""
        n, bad = _i32(), _i64()
        st = lib.ftp_check_guards(self.h, C.byref(n), C.byref(bad), _stream(stream))
        if st != OK:
            e = FtpError(st, lib.ftp_last_error().decode())
            e.bad_offset = bad.value
            raise e
        return n.value

    def ftp_check_device_status(self, stream=None):
        _check(lib.ftp_check_device_status(self.h, _stream(stream)))

    def ftp_debug_set_device_status(self, code, stream=None):
        _check(lib.ftp_debug_set_device_status(self.h, int(code), _stream(stream)))

    def ftp_trace_enable(self, on):
        _check(lib.ftp_trace_enable(self.h, int(on)))

    def ftp_trace_read(self, max_records=65536):
        buf = (TraceRec * max_records)()
        n = _i32()
        _check(lib.ftp_trace_read(self.h, buf, max_records, C.byref(n)))
        return [dict(kernel=ftp_kernel_name(r.kernel), unit=r.unit, op=r.op, backward=r.backward, ms=r.ms,
                     bytes=r.bytes, flops=r.flops) for r in buf[:min(n.value, max_records)]]

    def ftp_launch_count(self):
        n = _i64()
        _check(lib.ftp_launch_count(self.h, C.byref(n)))
        return n.value

    # -- marshalling helpers (no arithmetic) --
    def load_params(self, per_op_params, per_op_state=None):
        """Scatter per-op float32 arrays (canonical order) into the unit tensors."""
        for u in range(self.L):
            parts = [a.reshape(-1) for l, arrs in zip(self.layers, per_op_params) if l.unit == u for a in arrs]
            if parts:
                self.ftp_set_tensor(T_WEIGHTS, u, np.concatenate(parts).astype(np.float32))
            if per_op_state is not None:
                parts = [a.reshape(-1) for l, arrs in zip(self.layers, per_op_state) if l.unit == u for a in arrs]
                if parts:
                    self.ftp_set_tensor(T_STATE, u, np.concatenate(parts).astype(np.float32))


__all__ = ["Model", "FtpError", "LayerDesc", "ModelCfg", "TraceRec", "ftp_estimate_capacity", "ftp_choose_partition",
           "ftp_redistribution_plan", "ftp_recovery_plan", "FailedStage", "SRC_LOCAL", "SRC_STAGE", "SRC_REPLICA", "SRC_CENTRAL", "ftp_workspace_bytes", "ftp_kernel_name", "ftp_conv_wgrad_static", "layer_array", "model_cfg", "lib",
           "T_WEIGHTS", "T_GRADS", "T_MOMENTUM", "T_STATE", "FP32", "BF16", "LIB_PATH"]
