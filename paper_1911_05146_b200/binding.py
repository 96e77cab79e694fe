"""ctypes binding of libhpf.so: same names as the C ABI, argument marshalling only."""
import ctypes as C
import os

from . import build as _build

CONV, BNRELU, ADD, MAXPOOL, HEAD, BN, RELU = 1, 2, 3, 4, 5, 6, 7
OPT_GRAPH, OPT_CONV_PATH, OPT_SINGLE_STREAM, OPT_KEEP_MESSAGES, OPT_FUSE_ADD, OPT_PDL, OPT_WGRAD_PASSES, OPT_FUSE_BN, OPT_CELL_TIMES, OPT_BN_CLUSTER, OPT_CELL_CTAS, OPT_PDL_LATE_FROM, OPT_STAGE_LANES, OPT_WGRAD_DIRECT = 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14


class HpfError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"hpf status {status}: {text}")
        self.status = status


class _Op(C.Structure):
    _fields_ = [("kind", C.c_int32), ("src0", C.c_int32), ("src1", C.c_int32), ("c_in", C.c_int32),
                ("c_out", C.c_int32), ("ksize", C.c_int32), ("stride", C.c_int32), ("pad", C.c_int32),
                ("eps", C.c_float)]


_lib = None
_vp, _i32, _i64, _f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
_pi32, _pi64 = C.POINTER(C.c_int32), C.POINTER(C.c_int64)

# name -> argtypes; every function returns int except the two string getters
_SIGNATURES = {
    "hpf_model_create": [C.POINTER(_Op), _i32, _pi32, _pi32, _i32, _i32, C.POINTER(_vp)],
    "hpf_model_destroy": [_vp],
    "hpf_set_option": [_vp, _i32, _i32],
    "hpf_num_ops": [_vp, _pi32],
    "hpf_num_partitions": [_vp, _pi32],
    "hpf_num_stream_slots": [_vp, _pi32],
    "hpf_num_params": [_vp, _pi64],
    "hpf_param_layout": [_vp, _i32, _pi64, _pi64, _pi64, _pi64],
    "hpf_op_shape": [_vp, _i32, _pi32],
    "hpf_partition_of_op": [_vp, _i32, _pi32],
    "hpf_partition_range": [_vp, _i32, _pi32, _pi32],
    "hpf_microbatch_range": [_vp, _i32, _pi32, _pi32],
    "hpf_boundary_count": [_vp, _i32, _pi32],
    "hpf_boundary_desc": [_vp, _i32, _i32, _pi32, _pi32],
    "hpf_schedule_tick": [_vp, _i32, _i32, _pi32, _pi32],
    "hpf_estimate_op_costs": [C.POINTER(_Op), _i32, _pi32, C.POINTER(C.c_double)],
    "hpf_balance_cuts": [C.POINTER(C.c_double), _i32, _i32, _pi32],
    "hpf_workspace_bytes": [_vp, C.POINTER(C.c_size_t)],
    "hpf_bind": [_vp, _vp, _vp, _vp, _vp, C.c_size_t, C.POINTER(_vp), _i32],
    "hpf_forward": [_vp, _vp, _vp],
    "hpf_backward": [_vp],
    "hpf_forward_backward": [_vp, _vp, _vp],
    "hpf_prepare_partition": [_vp, _i32],
    "hpf_forward_cell": [_vp, _i32, _i32, _vp, _vp],
    "hpf_backward_cell": [_vp, _i32, _i32],
    "hpf_join_partition": [_vp, _i32],
    "hpf_partition_param_range": [_vp, _i32, _pi64, _pi64],
    "hpf_backward_message_count": [_vp, _i32, _pi32],
    "hpf_backward_message_desc": [_vp, _i32, _i32, _pi32, _pi32],
    "hpf_grad_average": [_vp],
    "hpf_loss": [_vp, C.POINTER(_f32)],
    "hpf_step_host": [_vp, _vp, _vp, C.POINTER(_f32)],
    "hpf_synchronize": [_vp, _i32],
    "hpf_tensor_ptr": [_vp, _i32, _i32, _i32, C.POINTER(_vp), _pi32],
    "hpf_message_ptr": [_vp, _i32, _i32, _i32, _i32, C.POINTER(_vp)],
    "hpf_loss_slots_ptr": [_vp, C.POINTER(_vp)],
    "hpf_sgd_momentum_step": [_vp, _vp, _f32, _f32, _f32],
    "hpf_sgd_momentum_flat": [_vp, _vp, _vp, _vp, _i32, _i64, _f32, _f32, _f32, _vp],
    "hpf_launch_count": [_vp, _pi64],
    "hpf_bnrelu_status": [_vp, _pi32],
    "hpf_step_bytes": [_vp, C.POINTER(C.c_double)],
    "hpf_cell_times": [_vp, _i32, _pi64],
    "hpf_conv_path_counts": [_vp, _pi64, _pi64],
    "hpf_conv_scratch_bytes": [_i32] * 8 + [C.POINTER(C.c_size_t)],
    "hpf_conv_prepare_weights": [_vp, _vp, _i32, _i32, _i32, _vp],
    "hpf_conv_fwd": [_vp, _vp, _vp, _vp] + [_i32] * 9 + [_vp, _vp],
    "hpf_conv_dgrad": [_vp, _vp, _vp, _vp] + [_i32] * 9 + [_vp, _vp],
    "hpf_conv_wgrad": [_vp, _vp, _vp] + [_i32] * 9 + [_vp, _vp],
    "hpf_bnrelu_scratch_bytes": [_i64, _i32, C.POINTER(C.c_size_t)],
    "hpf_bnrelu_fwd": [_vp, _vp, _vp, _f32, _vp, _vp, _i64, _i32, _vp, _vp],
    "hpf_bnrelu_bwd": [_vp] * 7 + [_i32, _vp, _vp, _i64, _i32, _vp, _vp],
    "hpf_grad_average_flat": [_vp, _vp, _i32, _i64, _vp],
    "hpf_bnrelu_fwd_static": [_vp, _vp, _vp, _f32, _vp, _vp, _i64, _i32, _vp],
    "hpf_static_scratch_bytes": [C.POINTER(C.c_size_t)],
}
EXPORTS = sorted(list(_SIGNATURES) + ["hpf_strerror", "hpf_last_error"])


def lib():
    """Loads (building if stale) the CUDA library.  Fails loudly if it cannot be built or loaded."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        for name, args in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = C.c_int
        L.hpf_strerror.argtypes = [C.c_int]
        L.hpf_strerror.restype = C.c_char_p
        L.hpf_last_error.argtypes = []
        L.hpf_last_error.restype = C.c_char_p
        _lib = L
    return _lib


def _check(status):
    if status != 0:
        L = lib()
        raise HpfError(status, f"{L.hpf_strerror(status).decode()} ({L.hpf_last_error().decode()})")


def _ptr(t):
    """Device (or pinned host) pointer of a torch tensor, or a raw integer address."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _op_array(ops):
    arr = (_Op * len(ops))()
    for i, o in enumerate(ops):
        arr[i] = _Op(*[int(v) for v in o[:8]], float(o[8]))
    return arr


def estimate_op_costs(ops, microbatch_shape):
    """Modelled microseconds (forward + backward chain) per op for one micro-batch of shape (b, H, W, C)."""
    out = (C.c_double * len(ops))()
    _check(lib().hpf_estimate_op_costs(_op_array(ops), len(ops), (_i32 * 4)(*microbatch_shape), out))
    return list(out)


def balance_cuts(costs, n_partitions):
    """Cut points minimising the largest partition cost."""
    cuts = (_i32 * max(n_partitions - 1, 1))()
    _check(lib().hpf_balance_cuts((C.c_double * len(costs))(*costs), len(costs), n_partitions, cuts))
    return list(cuts[:n_partitions - 1])


class Model:
    """Owns an hpf_model handle.  `ops` are tuples (kind, src0, src1, c_in, c_out, ksize, stride, pad, eps)."""

    def __init__(self, ops, in_shape, cuts, n_microbatches):
        arr = (_Op * len(ops))()
        for i, o in enumerate(ops):
            arr[i] = _Op(*[int(v) for v in o[:8]], float(o[8]))
        self._h = _vp()
        self._keep = []
        cuts = list(cuts)
        _check(lib().hpf_model_create(arr, len(ops), (_i32 * 4)(*in_shape), (_i32 * max(len(cuts), 1))(*cuts),
                                      len(cuts), n_microbatches, C.byref(self._h)))
        self.n_ops = len(ops)
        self.in_shape = tuple(in_shape)
        self.M = n_microbatches

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().hpf_model_destroy(self._h)
            self._h = _vp()

    __del__ = close

    # ---- options and bookkeeping
    def set_option(self, option, value):
        _check(lib().hpf_set_option(self._h, option, value))

    def num_params(self):
        g = _i64(); _check(lib().hpf_num_params(self._h, C.byref(g))); return g.value

    def num_partitions(self):
        p = _i32(); _check(lib().hpf_num_partitions(self._h, C.byref(p))); return p.value

    def num_stream_slots(self):
        s = _i32(); _check(lib().hpf_num_stream_slots(self._h, C.byref(s))); return s.value

    def param_layout(self, op):
        a, b, c, d = _i64(), _i64(), _i64(), _i64()
        _check(lib().hpf_param_layout(self._h, op, C.byref(a), C.byref(b), C.byref(c), C.byref(d)))
        return a.value, b.value, c.value, d.value

    def op_shape(self, op):
        s = (_i32 * 3)(); _check(lib().hpf_op_shape(self._h, op, s)); return tuple(s)

    def partition_of_op(self, op):
        p = _i32(); _check(lib().hpf_partition_of_op(self._h, op, C.byref(p))); return p.value

    def partition_range(self, p):
        a, b = _i32(), _i32(); _check(lib().hpf_partition_range(self._h, p, C.byref(a), C.byref(b))); return a.value, b.value

    def microbatch_range(self, m):
        a, b = _i32(), _i32(); _check(lib().hpf_microbatch_range(self._h, m, C.byref(a), C.byref(b))); return a.value, b.value

    def boundary_count(self, cut):
        n = _i32(); _check(lib().hpf_boundary_count(self._h, cut, C.byref(n))); return n.value

    def boundary_desc(self, cut, i):
        t = _i32(); s = (_i32 * 4)()
        _check(lib().hpf_boundary_desc(self._h, cut, i, C.byref(t), s)); return t.value, tuple(s)

    def schedule_tick(self, p, m):
        a, b = _i32(), _i32(); _check(lib().hpf_schedule_tick(self._h, p, m, C.byref(a), C.byref(b))); return a.value, b.value

    # ---- device resources
    def workspace_bytes(self):
        n = C.c_size_t(); _check(lib().hpf_workspace_bytes(self._h, C.byref(n))); return n.value

    def bind(self, params, grad_slots, grad_avg, workspace, streams):
        """All arguments are torch CUDA tensors (kept alive by this object); streams are torch.cuda.Stream."""
        self._keep = [params, grad_slots, grad_avg, workspace, list(streams)]
        handles = (_vp * len(streams))(*[_stream(s) for s in streams])
        ws_bytes = workspace.numel() * workspace.element_size()
        _check(lib().hpf_bind(self._h, _ptr(params), _ptr(grad_slots), _ptr(grad_avg), _ptr(workspace), ws_bytes,
                              handles, len(streams)))

    # ---- the step
    def forward(self, x, labels):
        self._keep_inputs = (x, labels)
        _check(lib().hpf_forward(self._h, _ptr(x), _ptr(labels)))

    def backward(self):
        _check(lib().hpf_backward(self._h))

    # ---- one cell at a time (stage-per-GPU runs) ----
    def prepare_partition(self, p):
        _check(lib().hpf_prepare_partition(self._h, int(p)))

    def forward_cell(self, p, m, x=None, labels=None):
        self._keep_inputs = (x, labels) if x is not None or labels is not None else getattr(self, "_keep_inputs", None)
        _check(lib().hpf_forward_cell(self._h, int(p), int(m), _ptr(x), _ptr(labels)))

    def backward_cell(self, p, m):
        _check(lib().hpf_backward_cell(self._h, int(p), int(m)))

    def join_partition(self, p):
        _check(lib().hpf_join_partition(self._h, int(p)))

    def partition_param_range(self, p):
        a, b = _i64(), _i64(); _check(lib().hpf_partition_param_range(self._h, int(p), C.byref(a), C.byref(b))); return a.value, b.value

    def backward_messages(self, cut):
        """Ops whose gradient buffers partition cut+1 hands down across `cut`, with their shapes (b, H, W, C)."""
        n = _i32(); _check(lib().hpf_backward_message_count(self._h, int(cut), C.byref(n)))
        out = []
        for j in range(n.value):
            op = _i32(); shape = (_i32 * 4)()
            _check(lib().hpf_backward_message_desc(self._h, int(cut), j, C.byref(op), shape))
            out.append((op.value, tuple(shape)))
        return out

    def forward_backward(self, x, labels):
        self._keep_inputs = (x, labels)
        _check(lib().hpf_forward_backward(self._h, _ptr(x), _ptr(labels)))

    def grad_average(self):
        _check(lib().hpf_grad_average(self._h))

    def sgd_momentum_step(self, velocity, lr, momentum=0.0, weight_decay=0.0):
        _check(lib().hpf_sgd_momentum_step(self._h, _ptr(velocity), lr, momentum, weight_decay))

    def loss(self):
        v = _f32(); _check(lib().hpf_loss(self._h, C.byref(v))); return v.value

    def step_host(self, h_x, h_labels):
        v = _f32(); _check(lib().hpf_step_host(self._h, _ptr(h_x), _ptr(h_labels), C.byref(v))); return v.value

    def synchronize(self, timeout_ms=0):
        _check(lib().hpf_synchronize(self._h, timeout_ms))

    # ---- inspection
    def tensor_ptr(self, op, m, want_grad=False):
        p = _vp(); s = (_i32 * 4)()
        _check(lib().hpf_tensor_ptr(self._h, op, m, int(want_grad), C.byref(p), s)); return p.value, tuple(s)

    def message_ptr(self, cut, i, m, want_grad=False):
        p = _vp(); _check(lib().hpf_message_ptr(self._h, cut, i, m, int(want_grad), C.byref(p))); return p.value

    def loss_slots_ptr(self):
        p = _vp(); _check(lib().hpf_loss_slots_ptr(self._h, C.byref(p))); return p.value

    def cell_times(self, phase):
        """ns timestamps [p][m] = (start, end) of every cell of the last forward (0) / backward (1)."""
        P = self.num_partitions()
        buf = (_i64 * (P * self.M * 2))(); _check(lib().hpf_cell_times(self._h, int(phase), buf))
        return [[(buf[(p * self.M + m) * 2], buf[(p * self.M + m) * 2 + 1]) for m in range(self.M)] for p in range(P)]

    def step_bytes(self):
        v = C.c_double(); _check(lib().hpf_step_bytes(self._h, C.byref(v))); return v.value

    def launch_count(self):
        n = _i64(); _check(lib().hpf_launch_count(self._h, C.byref(n))); return n.value

    def conv_path_counts(self):
        a, b = _i64(), _i64(); _check(lib().hpf_conv_path_counts(self._h, C.byref(a), C.byref(b))); return a.value, b.value


# ---- single kernels on caller buffers -------------------------------------------------------------
def bnrelu_status(scratch):
    """True if a bounded wait of a single-op BN call on this scratch gave up (the scratch head must then be zeroed again)."""
    v = _i32(); _check(lib().hpf_bnrelu_status(_ptr(scratch), C.byref(v))); return bool(v.value)


def conv_scratch_bytes(N, H, W, Cc, K, R, stride, pad):
    n = C.c_size_t(); _check(lib().hpf_conv_scratch_bytes(N, H, W, Cc, K, R, stride, pad, C.byref(n))); return n.value


def conv_prepare_weights(w, wprep, Cc, K, R, stream=None):
    _check(lib().hpf_conv_prepare_weights(_ptr(w), _ptr(wprep), Cc, K, R, _stream(stream)))


def conv_fwd(x, w, wprep, y, N, H, W, Cc, K, R, stride, pad, path, scratch, stream=None):
    _check(lib().hpf_conv_fwd(_ptr(x), _ptr(w), _ptr(wprep), _ptr(y), N, H, W, Cc, K, R, stride, pad, path, _ptr(scratch),
                              _stream(stream)))


def conv_dgrad(dy, w, wprep, dx, N, H, W, Cc, K, R, stride, pad, path, scratch, stream=None):
    _check(lib().hpf_conv_dgrad(_ptr(dy), _ptr(w), _ptr(wprep), _ptr(dx), N, H, W, Cc, K, R, stride, pad, path,
                                _ptr(scratch), _stream(stream)))


def conv_wgrad(x, dy, dw, N, H, W, Cc, K, R, stride, pad, path, scratch, stream=None):
    _check(lib().hpf_conv_wgrad(_ptr(x), _ptr(dy), _ptr(dw), N, H, W, Cc, K, R, stride, pad, path, _ptr(scratch), _stream(stream)))


def bnrelu_scratch_bytes(rows, Cc):
    n = C.c_size_t(); _check(lib().hpf_bnrelu_scratch_bytes(rows, Cc, C.byref(n))); return n.value


def bnrelu_fwd(x, gamma, beta, eps, y, stats, rows, Cc, scratch, stream=None):
    _check(lib().hpf_bnrelu_fwd(_ptr(x), _ptr(gamma), _ptr(beta), eps, _ptr(y), _ptr(stats), rows, Cc, _ptr(scratch), _stream(stream)))


def bnrelu_bwd(x, dy, gamma, beta, stats, dx, addend, accumulate, dgamma, dbeta, rows, Cc, scratch, stream=None):
    _check(lib().hpf_bnrelu_bwd(_ptr(x), _ptr(dy), _ptr(gamma), _ptr(beta), _ptr(stats), _ptr(dx), _ptr(addend),
                                int(accumulate), _ptr(dgamma), _ptr(dbeta), rows, Cc, _ptr(scratch), _stream(stream)))


def grad_average_flat(slots, out, M, G, stream=None):
    _check(lib().hpf_grad_average_flat(_ptr(slots), _ptr(out), M, G, _stream(stream)))


def sgd_momentum_flat(slots, grad_avg, params, velocity, M, G, lr, momentum=0.0, weight_decay=0.0, stream=None):
    _check(lib().hpf_sgd_momentum_flat(_ptr(slots), _ptr(grad_avg) if grad_avg is not None else None, _ptr(params), _ptr(velocity),
                                       M, G, lr, momentum, weight_decay, _stream(stream)))


def bnrelu_fwd_static(x, gamma, beta, eps, y, stats, rows, Cc, stream=None):
    """BN+ReLU forward on the library's built-in scratch: for callers that cannot allocate (see hpf.h)."""
    _check(lib().hpf_bnrelu_fwd_static(_ptr(x), _ptr(gamma), _ptr(beta), eps, _ptr(y), _ptr(stats), rows, Cc, _stream(stream)))


def static_scratch_bytes():
    n = C.c_size_t(); _check(lib().hpf_static_scratch_bytes(C.byref(n))); return n.value
