"""Thin ctypes binding over libmpt.so (the C ABI declared in include/mpt.h).

Argument marshalling only: every arithmetic step runs in the CUDA library.  PyTorch
is used for device memory (the workspace and the tensors handed in) and streams.
There is no fallback: if the shared library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# MPT_LIB: another build of the library to load instead (comparing two builds in one session)
LIB_PATH = os.environ.get("MPT_LIB") or os.path.join(_HERE, "libmpt.so")

OK = 0
ERR = {-1: "MPT_ERR_INVALID_ARG", -2: "MPT_ERR_SHAPE", -3: "MPT_ERR_STATE", -4: "MPT_ERR_WORKSPACE",
       -5: "MPT_ERR_CUDA", -6: "MPT_ERR_TIMEOUT", -7: "MPT_ERR_INTERNAL"}
OP_FWD, OP_DGRAD, OP_WGRAD = 0, 1, 2
GEMM_RELU, GEMM_FORCE_SIMT, GEMM_FORCE_TC, GEMM_FORCE_PAIR, GEMM_FORCE_PAIR512 = 1, 2, 4, 8, 16
GEMM_FORCE_SPLIT2, GEMM_FORCE_SPLIT4 = 32, 64
T_W16, T_GRAD16, T_ACT16, T_DACT16, T_MOMENTUM32, T_MASTER32, T_STATE2_32 = range(7)
OPT_SGD, OPT_NESTEROV, OPT_ADAGRAD, OPT_ADAM = 0, 1, 2, 3

# every symbol include/mpt.h declares
EXPORTS = ["mpt_workspace_bytes", "mpt_create", "mpt_workspace_bytes_opt", "mpt_create_opt", "mpt_set_state2",
           "mpt_get_adam_products", "mpt_set_adam_products", "mpt_get_grad_norm", "mpt_update_flat_opt", "mpt_set_master", "mpt_forward", "mpt_backward_scaled",
           "mpt_step", "mpt_get_master", "mpt_train_step_host", "mpt_stage_batch_host",
           "mpt_train_step_staged", "mpt_set_scale", "mpt_set_lr", "mpt_set_dynamic_scale", "mpt_get_scale",
           "mpt_get_tensor", "mpt_set_grad", "mpt_set_momentum", "mpt_launch_count", "mpt_profile",
           "mpt_profile_read", "mpt_last_error",
           "mpt_destroy", "mpt_gemm_f16", "mpt_gemm_f16_ws", "mpt_gemm_workspace_bytes", "mpt_recast", "mpt_grad_nonfinite", "mpt_update_flat",
           "mpt_softmax_ce", "mpt_softmax_ce_static", "mpt_version",
           "mpt_selftest_wait_timeout", "mpt_selftest_wait_timeout_ctx", "mpt_sm_clock_probe",
           "mpt_lstm_workspace_bytes", "mpt_lstm_create", "mpt_lstm_set_params", "mpt_lstm_train_step", "mpt_lstm_get_tensor",
           "mpt_lstm_set_dynamic_scale", "mpt_lstm_get_scale", "mpt_lstm_last_error", "mpt_lstm_destroy",
           "mpt_lstm_forward", "mpt_lstm_backward", "mpt_lstm_cell_forward", "mpt_lstm_cell_backward", "mpt_bias_grad",
           "mpt_add_f16",
           "mpt_dp_shard", "mpt_dp_step_flat", "mpt_dp_alloc", "mpt_dp_free", "mpt_dp_export", "mpt_dp_open", "mpt_dp_close",
           "mpt_dp_layout_of", "mpt_dp_attach", "mpt_dp_step_flat_opt", "mpt_dp_norm_flat", "mpt_dp_norm",
           "mpt_workspace_bytes_dp", "mpt_create_dp", "mpt_state_range", "mpt_dp_overlap_events", "mpt_dp_overlap_attach",
           "mpt_dp_reduce_async"]


class MptError(RuntimeError):
    def __init__(self, code, msg=""):
        self.code = code
        super().__init__("%s (%d) %s" % (ERR.get(code, "MPT_ERR_?"), code, msg))


class LayerDesc(C.Structure):
    _fields_ = [("in_features", C.c_int32), ("out_features", C.c_int32), ("relu", C.c_int32)]


class Optimizer(C.Structure):
    """mpt_optimizer: kind (OPT_*), lr, momentum (or Adam beta1), beta2, eps, weight_decay, clip_norm."""
    _fields_ = [("kind", C.c_int32), ("lr", C.c_float), ("momentum", C.c_float), ("beta2", C.c_float),
                ("eps", C.c_float), ("weight_decay", C.c_float), ("clip_norm", C.c_float)]


class LstmDesc(C.Structure):
    """mpt_lstm_desc: T steps, B rows per step, input width I, H cells, projection width P."""
    _fields_ = [("T", C.c_int32), ("B", C.c_int32), ("I", C.c_int32), ("H", C.c_int32), ("P", C.c_int32)]


_LSTM_FIELDS = ["Wg16", "bias16", "Wp16", "xr", "c", "h", "acts", "dr_ext", "dxr", "drtot", "dG", "dh", "dc", "dWg16", "dWp16",
                "dbias16", "bias_parts", "nonfinite_flag", "status_dev"]


class LstmTensors(C.Structure):
    """mpt_lstm_tensors: device pointers of every tensor of the layer (see include/mpt.h)."""
    _fields_ = [(name, C.c_void_p) for name in _LSTM_FIELDS] + [("splitk_ws", C.c_void_p), ("splitk_ws_bytes", C.c_size_t)]


_lib = None


class DpLayout(C.Structure):
    _fields_ = [("g16_offset", C.c_size_t), ("w16_offset", C.c_size_t), ("flags_offset", C.c_size_t), ("n", C.c_size_t)]


def lib() -> C.CDLL:
    """Load libmpt.so; raises if it has not been built (python -m paper_1710_03740_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("CUDA library %s not found: run `python -m paper_1710_03740_b200.build`" % LIB_PATH)
    L = C.CDLL(LIB_PATH)
    vp, i32, u32, f32, sz = C.c_void_p, C.c_int, C.c_uint, C.c_float, C.c_size_t
    L.mpt_workspace_bytes.argtypes = [C.POINTER(LayerDesc), i32, i32, i32, C.POINTER(sz)]
    L.mpt_create.argtypes = [C.POINTER(LayerDesc), i32, f32, f32, f32, i32, vp, sz, vp, C.POINTER(vp)]
    L.mpt_workspace_bytes_opt.argtypes = [C.POINTER(LayerDesc), i32, i32, C.POINTER(Optimizer), C.POINTER(sz)]
    L.mpt_create_opt.argtypes = [C.POINTER(LayerDesc), i32, f32, C.POINTER(Optimizer), i32, vp, sz, vp, C.POINTER(vp)]
    L.mpt_workspace_bytes_dp.argtypes = [C.POINTER(LayerDesc), i32, i32, C.POINTER(Optimizer), i32, i32, C.POINTER(sz)]
    L.mpt_create_dp.argtypes = [C.POINTER(LayerDesc), i32, f32, C.POINTER(Optimizer), i32, i32, i32, vp, sz, vp, C.POINTER(vp)]
    L.mpt_state_range.argtypes = [vp, i32, C.POINTER(sz), C.POINTER(sz)]
    L.mpt_dp_overlap_events.argtypes = [vp, vp]
    L.mpt_dp_overlap_attach.argtypes = [vp, vp, vp, sz]
    L.mpt_dp_reduce_async.argtypes = [vp]
    L.mpt_set_state2.argtypes = [vp, i32, vp, sz]
    L.mpt_get_adam_products.argtypes = [vp, C.POINTER(f32), C.POINTER(f32)]
    L.mpt_set_adam_products.argtypes = [vp, f32, f32]
    L.mpt_update_flat_opt.argtypes = [C.POINTER(Optimizer), vp, vp, vp, vp, vp, sz, f32, f32, f32, i32, vp, vp, vp]
    L.mpt_get_grad_norm.argtypes = [vp, C.POINTER(f32), C.POINTER(f32)]
    L.mpt_set_master.argtypes = [vp, i32, vp, sz]
    L.mpt_forward.argtypes = [vp, vp, i32]
    L.mpt_backward_scaled.argtypes = [vp, vp, C.POINTER(f32)]
    L.mpt_step.argtypes = [vp, C.POINTER(i32)]
    L.mpt_get_master.argtypes = [vp, i32, vp, sz]
    L.mpt_train_step_host.argtypes = [vp, vp, vp, i32, C.POINTER(f32), C.POINTER(i32)]
    L.mpt_stage_batch_host.argtypes = [vp, vp, vp, i32, vp]
    L.mpt_train_step_staged.argtypes = [vp, C.POINTER(f32), C.POINTER(i32)]
    L.mpt_set_scale.argtypes = [vp, f32]
    L.mpt_set_lr.argtypes = [vp, f32]
    L.mpt_set_dynamic_scale.argtypes = [vp, i32, i32, f32, f32]
    L.mpt_get_scale.argtypes = [vp, C.POINTER(f32)]
    L.mpt_get_tensor.argtypes = [vp, i32, i32, vp, sz]
    L.mpt_set_grad.argtypes = [vp, i32, vp, sz]
    L.mpt_set_momentum.argtypes = [vp, i32, vp, sz]
    L.mpt_launch_count.argtypes = [vp, C.POINTER(C.c_longlong)]
    L.mpt_profile.argtypes = [vp, i32]
    L.mpt_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_longlong)]
    L.mpt_last_error.argtypes = [vp]
    L.mpt_last_error.restype = C.c_char_p
    L.mpt_destroy.argtypes = [vp]
    L.mpt_destroy.restype = None
    L.mpt_gemm_f16.argtypes = [i32, i32, i32, i32, vp, i32, vp, i32, vp, i32, u32, vp, i32, vp, vp, vp]
    L.mpt_gemm_f16_ws.argtypes = [i32, i32, i32, i32, vp, i32, vp, i32, vp, i32, u32, vp, i32, vp, vp, vp, sz, vp]
    L.mpt_gemm_workspace_bytes.argtypes = [i32, i32, i32, i32, C.POINTER(sz)]
    L.mpt_recast.argtypes = [vp, vp, sz, vp]
    L.mpt_grad_nonfinite.argtypes = [vp, sz, f32, vp, vp]
    L.mpt_update_flat.argtypes = [vp, vp, vp, vp, sz, f32, f32, f32, i32, i32, vp, vp]
    L.mpt_softmax_ce.argtypes = [vp, i32, vp, i32, i32, f32, vp, i32, vp, vp, vp, vp, vp]
    L.mpt_softmax_ce_static.argtypes = [vp, i32, vp, i32, i32, f32, vp, i32, vp, vp, vp, vp]
    L.mpt_sm_clock_probe.argtypes = [u32, vp, vp]
    L.mpt_lstm_workspace_bytes.argtypes = [C.POINTER(LstmDesc), C.POINTER(Optimizer), C.POINTER(sz)]
    L.mpt_lstm_create.argtypes = [C.POINTER(LstmDesc), f32, C.POINTER(Optimizer), vp, sz, vp, C.POINTER(vp)]
    L.mpt_lstm_set_params.argtypes = [vp, vp, vp, vp]
    L.mpt_lstm_train_step.argtypes = [vp, vp, vp, C.POINTER(f32), C.POINTER(i32)]
    L.mpt_lstm_get_tensor.argtypes = [vp, i32, vp, sz]
    L.mpt_lstm_set_dynamic_scale.argtypes = [vp, i32, i32, f32, f32]
    L.mpt_lstm_get_scale.argtypes = [vp, C.POINTER(f32)]
    L.mpt_lstm_last_error.argtypes = [vp]
    L.mpt_lstm_last_error.restype = C.c_char_p
    L.mpt_lstm_destroy.argtypes = [vp]
    L.mpt_lstm_destroy.restype = None
    L.mpt_selftest_wait_timeout.argtypes = [u32, vp, vp]
    L.mpt_selftest_wait_timeout_ctx.argtypes = [vp, u32]
    L.mpt_lstm_forward.argtypes = [C.POINTER(LstmDesc), C.POINTER(LstmTensors), vp]
    L.mpt_lstm_backward.argtypes = [C.POINTER(LstmDesc), C.POINTER(LstmTensors), vp]
    L.mpt_lstm_cell_forward.argtypes = [i32, i32, i32, vp, i32, vp, i32, vp, vp, i32, vp, i32, vp, i32, vp, i32, u32, vp, vp]
    L.mpt_lstm_cell_backward.argtypes = [i32, i32, vp, i32, vp, i32, vp, i32, vp, i32, vp, i32, vp, i32, vp, i32, vp]
    L.mpt_bias_grad.argtypes = [vp, sz, i32, i32, vp, vp, vp, vp]
    L.mpt_add_f16.argtypes = [vp, i32, vp, i32, vp, i32, i32, i32, vp]
    L.mpt_dp_shard.argtypes = [sz, i32, i32, C.POINTER(sz), C.POINTER(sz)]
    L.mpt_dp_step_flat.argtypes = [vp, vp, vp, vp, vp, sz, i32, i32, f32, f32, f32, vp, vp]
    L.mpt_dp_step_flat_opt.argtypes = [C.POINTER(Optimizer), vp, vp, vp, vp, vp, vp, sz, i32, i32, f32, f32, f32, vp, vp, vp, vp]
    L.mpt_dp_norm_flat.argtypes = [vp, sz, i32, i32, f32, vp, vp, vp]
    L.mpt_dp_norm.argtypes = [vp]
    L.mpt_dp_alloc.argtypes = [sz, C.POINTER(vp)]
    L.mpt_dp_free.argtypes = [vp]
    L.mpt_dp_export.argtypes = [vp, vp]
    L.mpt_dp_open.argtypes = [vp, C.POINTER(vp)]
    L.mpt_dp_close.argtypes = [vp]
    L.mpt_dp_layout_of.argtypes = [vp, C.POINTER(DpLayout)]
    L.mpt_dp_attach.argtypes = [vp, i32, i32, vp, vp, vp]
    L.mpt_version.restype = C.c_char_p
    L.mpt_version.argtypes = []
    _lib = L
    return L


def _check(code, ctx=None):
    if code != OK:
        msg = ""
        if ctx:
            msg = lib().mpt_last_error(ctx).decode()
        raise MptError(code, msg)


def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _hptr(a):
    """Host pointer of a numpy array or a CPU torch tensor."""
    if isinstance(a, np.ndarray):
        return C.c_void_p(a.ctypes.data)
    return C.c_void_p(a.data_ptr())


def _layer_array(layers):
    arr = (LayerDesc * len(layers))()
    for k, (i, o, r) in enumerate(layers):
        arr[k].in_features, arr[k].out_features, arr[k].relu = int(i), int(o), int(r)
    return arr


def mpt_workspace_bytes(layers, max_batch, use_momentum) -> int:
    out = C.c_size_t(0)
    _check(lib().mpt_workspace_bytes(_layer_array(layers), len(layers), int(max_batch), int(bool(use_momentum)),
                                     C.byref(out)))
    return int(out.value)


class Context:
    """One mpt_ctx over a torch-allocated workspace.  Method names follow the C calls."""

    def __init__(self, layers, S, lr, momentum=0.0, max_batch=1, device="cuda:0", stream=None, optimizer=None,
                 shareable=False, shard=None):
        """optimizer: an Optimizer struct; default SGD with the given lr and momentum.  shareable: take
        the workspace from the driver's allocator (a DeviceBuffer other processes can map) instead of
        torch's pool.  shard: (replicas, rank) - mpt_create_dp: FP32 state for that replica's shard only."""
        import torch
        self.layers = [(int(i), int(o), int(r)) for (i, o, r) in layers]
        self.device = torch.device(device)
        self.stream = stream
        opt = optimizer if optimizer is not None else Optimizer(OPT_SGD, float(lr), float(momentum), 0.0, 0.0, 0.0)
        self.optimizer = opt
        out = C.c_size_t(0)
        self.shard = (int(shard[0]), int(shard[1])) if shard else None
        if self.shard:
            _check(lib().mpt_workspace_bytes_dp(_layer_array(self.layers), len(self.layers), int(max_batch), C.byref(opt),
                                                self.shard[0], self.shard[1], C.byref(out)))
        else:
            _check(lib().mpt_workspace_bytes_opt(_layer_array(self.layers), len(self.layers), int(max_batch), C.byref(opt),
                                                 C.byref(out)))
        nbytes = int(out.value)
        with torch.cuda.device(self.device):
            if shareable:
                self.workspace = DeviceBuffer(nbytes + 256)
                base = self.workspace.ptr
                torch.cuda.synchronize()
            else:
                self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
                base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            self._ctx = C.c_void_p()
            if self.shard:
                _check(lib().mpt_create_dp(_layer_array(self.layers), len(self.layers), float(S), C.byref(opt),
                                           int(max_batch), self.shard[0], self.shard[1], C.c_void_p(self._ws_ptr), nbytes,
                                           _stream_ptr(stream), C.byref(self._ctx)))
            else:
                _check(lib().mpt_create_opt(_layer_array(self.layers), len(self.layers), float(S), C.byref(opt),
                                            int(max_batch), C.c_void_p(self._ws_ptr), nbytes, _stream_ptr(stream),
                                            C.byref(self._ctx)))
        self.workspace_bytes = nbytes
        self.batch = 0

    def close(self):
        if getattr(self, "_ctx", None):
            lib().mpt_destroy(self._ctx)
            self._ctx = None
            if isinstance(self.workspace, DeviceBuffer):
                self.workspace.close()

    def state_range(self, layer):
        """(first, count): the elements of the layer whose FP32 master and optimizer state live here."""
        first, count = C.c_size_t(0), C.c_size_t(0)
        _check(lib().mpt_state_range(self._ctx, int(layer), C.byref(first), C.byref(count)), self._ctx)
        return int(first.value), int(count.value)

    def dp_overlap_events(self):
        """Handles of this context's per-layer events (bytes) for the other replicas."""
        buf = (C.c_uint8 * ((len(self.layers) + 1) * DP_HANDLE_BYTES))()
        _check(lib().mpt_dp_overlap_events(self._ctx, buf), self._ctx)
        return bytes(buf)

    def dp_overlap_attach(self, peer_handles, rank):
        """peer_handles: list of R byte strings from dp_overlap_events (entry `rank` ignored)."""
        import torch
        R = len(peer_handles)
        lo, hi = mpt_dp_shard(self.dp_layout().n, R, rank)
        self._sum32 = torch.empty(max(hi - lo, 4), dtype=torch.float32, device=self.device)
        keep = [C.create_string_buffer(h, len(h)) if q != rank else None for q, h in enumerate(peer_handles)]
        tab = (C.c_void_p * R)(*[C.cast(k, C.c_void_p) if k is not None else None for k in keep])
        _check(lib().mpt_dp_overlap_attach(self._ctx, tab, _dptr(self._sum32), self._sum32.numel() * 4), self._ctx)

    def dp_reduce_async(self):
        _check(lib().mpt_dp_reduce_async(self._ctx), self._ctx)

    def dp_layout(self):
        out = DpLayout()
        _check(lib().mpt_dp_layout_of(self._ctx, C.byref(out)), self._ctx)
        return out

    def dp_norm(self):
        """Clipping in data-parallel mode: publish this replica's shard of the squared norm of the
        mean gradient (call on every replica after backward_scaled, order the replicas, then step)."""
        _check(lib().mpt_dp_norm(self._ctx), self._ctx)

    def dp_attach(self, R, rank, g16_peers, flag_peers, w16_peers):
        tab = lambda xs: (C.c_void_p * R)(*[_addr(x) for x in xs])
        _check(lib().mpt_dp_attach(self._ctx, int(R), int(rank), tab(g16_peers), tab(flag_peers), tab(w16_peers)), self._ctx)

    def __del__(self):
        try:                # at interpreter shutdown the module globals may already be gone
            self.close()
        except Exception:
            pass

    def set_master(self, layer, w32):
        w = np.ascontiguousarray(w32, dtype=np.float32)
        _check(lib().mpt_set_master(self._ctx, layer, _hptr(w), w.size), self._ctx)

    def get_master(self, layer):
        i, o, _ = self.layers[layer]
        # a context with FP32 state for its shard only fills in just that part (state_range): NaN elsewhere
        out = np.full((o, i), np.nan, dtype=np.float32) if self.shard else np.empty((o, i), dtype=np.float32)
        _check(lib().mpt_get_master(self._ctx, layer, _hptr(out), out.size), self._ctx)
        return out

    def forward(self, x_dev):
        """x_dev: torch float16 CUDA tensor [batch, in_1], contiguous; kept alive by the caller."""
        assert x_dev.is_cuda and x_dev.is_contiguous() and x_dev.element_size() == 2
        self.batch = int(x_dev.shape[0])
        _check(lib().mpt_forward(self._ctx, _dptr(x_dev), self.batch), self._ctx)

    def backward_scaled(self, labels_dev, want_loss=True):
        assert labels_dev.is_cuda and labels_dev.is_contiguous() and labels_dev.element_size() == 4
        if want_loss:
            loss = C.c_float(0.0)
            _check(lib().mpt_backward_scaled(self._ctx, _dptr(labels_dev), C.byref(loss)), self._ctx)
            return float(loss.value)
        _check(lib().mpt_backward_scaled(self._ctx, _dptr(labels_dev), None), self._ctx)
        return None

    def step(self, want_flag=True):
        if want_flag:
            flag = C.c_int(0)
            _check(lib().mpt_step(self._ctx, C.byref(flag)), self._ctx)
            return int(flag.value)
        _check(lib().mpt_step(self._ctx, None), self._ctx)
        return None

    def train_step_host(self, x_host, labels_host):
        """x_host: float16/uint16 [batch, in_1] host array (numpy or pinned torch); labels int32 [batch]."""
        batch = int(x_host.shape[0])
        loss, flag = C.c_float(0.0), C.c_int(0)
        _check(lib().mpt_train_step_host(self._ctx, _hptr(x_host), _hptr(labels_host), batch, C.byref(loss),
                                         C.byref(flag)), self._ctx)
        self.batch = batch
        return float(loss.value), int(flag.value)

    def stage_batch_host(self, x_host, labels_host, copy_stream):
        """Start the host-to-device copy of one batch on `copy_stream` (a torch.cuda.Stream)."""
        _check(lib().mpt_stage_batch_host(self._ctx, _hptr(x_host), _hptr(labels_host), int(x_host.shape[0]),
                                          C.c_void_p(copy_stream.cuda_stream)), self._ctx)

    def train_step_staged(self):
        loss, flag = C.c_float(0.0), C.c_int(0)
        _check(lib().mpt_train_step_staged(self._ctx, C.byref(loss), C.byref(flag)), self._ctx)
        return float(loss.value), int(flag.value)

    def set_scale(self, S):
        _check(lib().mpt_set_scale(self._ctx, float(S)), self._ctx)

    def set_dynamic_scale(self, enable, growth_interval=2000, min_scale=2.0 ** -14, max_scale=2.0 ** 24):
        _check(lib().mpt_set_dynamic_scale(self._ctx, int(bool(enable)), int(growth_interval), float(min_scale),
                                           float(max_scale)), self._ctx)

    def get_scale(self):
        S = C.c_float(0.0)
        _check(lib().mpt_get_scale(self._ctx, C.byref(S)), self._ctx)
        return float(S.value)

    def set_lr(self, lr):
        _check(lib().mpt_set_lr(self._ctx, float(lr)), self._ctx)

    def get_tensor(self, kind, layer):
        i, o, _ = self.layers[layer]
        if kind in (T_W16, T_GRAD16):
            out = np.empty((o, i), dtype=np.uint16)
        elif kind in (T_MOMENTUM32, T_MASTER32, T_STATE2_32):
            out = np.full((o, i), np.nan, dtype=np.float32) if self.shard else np.empty((o, i), dtype=np.float32)
        else:
            out = np.empty((self.batch, o), dtype=np.uint16)
        _check(lib().mpt_get_tensor(self._ctx, kind, layer, _hptr(out), out.nbytes), self._ctx)
        return out

    def set_grad(self, layer, g16):
        g = np.ascontiguousarray(g16)
        if g.dtype == np.float16:
            g = g.view(np.uint16)
        assert g.dtype == np.uint16
        _check(lib().mpt_set_grad(self._ctx, layer, _hptr(g), g.size), self._ctx)

    def set_momentum(self, layer, v):
        v = np.ascontiguousarray(v, dtype=np.float32)
        _check(lib().mpt_set_momentum(self._ctx, layer, _hptr(v), v.size), self._ctx)

    def profile(self, enable):
        _check(lib().mpt_profile(self._ctx, int(bool(enable))), self._ctx)

    def profile_read(self):
        """{class name: (milliseconds, algorithmic work, launches)} since profile(True)."""
        ms, work, n = (C.c_double * 4)(), (C.c_double * 4)(), (C.c_longlong * 4)()
        _check(lib().mpt_profile_read(self._ctx, ms, work, n), self._ctx)
        names = ("gemm", "update", "softmax", "other")
        return {names[k]: (float(ms[k]), float(work[k]), int(n[k])) for k in range(4)}

    def set_state2(self, layer, v):
        v = np.ascontiguousarray(v, dtype=np.float32)
        _check(lib().mpt_set_state2(self._ctx, layer, _hptr(v), v.size), self._ctx)

    def get_adam_products(self):
        a, b = C.c_float(0.0), C.c_float(0.0)
        _check(lib().mpt_get_adam_products(self._ctx, C.byref(a), C.byref(b)), self._ctx)
        return float(a.value), float(b.value)

    def get_grad_norm(self):
        """(norm of the unscaled gradients, clipping coefficient) of the last step."""
        a, b = C.c_float(0.0), C.c_float(0.0)
        _check(lib().mpt_get_grad_norm(self._ctx, C.byref(a), C.byref(b)), self._ctx)
        return float(a.value), float(b.value)

    def set_adam_products(self, b1t, b2t):
        _check(lib().mpt_set_adam_products(self._ctx, float(b1t), float(b2t)), self._ctx)

    def selftest_wait_timeout(self):
        """Makes a bounded device-side wait run out inside this context (1 ms limit): raises
        MptError(MPT_ERR_TIMEOUT) and leaves the context poisoned, as a real expiry would."""
        _check(lib().mpt_selftest_wait_timeout_ctx(self._ctx, 1000), self._ctx)

    def last_error(self) -> str:
        return lib().mpt_last_error(self._ctx).decode()

    def launch_count(self):
        n = C.c_longlong(0)
        _check(lib().mpt_launch_count(self._ctx, C.byref(n)), self._ctx)
        return int(n.value)


# ------------------------------------------------------------ stateless calls

def mpt_gemm_f16(op, M, N, K, A, lda, B, ldb, Cout, ldc, flags=0, mask=None, ldmask=0, nonfinite_flag=None,
                 status=None, stream=None):
    """Arguments are torch CUDA tensors (any 2-byte dtype) used as raw device pointers."""
    _check(lib().mpt_gemm_f16(op, M, N, K, _dptr(A), lda, _dptr(B), ldb, _dptr(Cout), ldc, flags, _dptr(mask), ldmask,
                              _dptr(nonfinite_flag), _dptr(status), _stream_ptr(stream)))


def mpt_gemm_workspace_bytes(op, M, N, K) -> int:
    out = C.c_size_t(0)
    _check(lib().mpt_gemm_workspace_bytes(op, M, N, K, C.byref(out)))
    return int(out.value)


def mpt_gemm_f16_ws(op, M, N, K, A, lda, B, ldb, Cout, ldc, flags=0, mask=None, ldmask=0, nonfinite_flag=None,
                    status=None, workspace=None, stream=None):
    """mpt_gemm_f16 with a scratch tensor (any dtype, 16-byte aligned) that permits split-K."""
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().mpt_gemm_f16_ws(op, M, N, K, _dptr(A), lda, _dptr(B), ldb, _dptr(Cout), ldc, flags, _dptr(mask), ldmask,
                                 _dptr(nonfinite_flag), _dptr(status), _dptr(workspace), nbytes, _stream_ptr(stream)))


def mpt_recast(w32, w16, n, stream=None):
    _check(lib().mpt_recast(_dptr(w32), _dptr(w16), n, _stream_ptr(stream)))


def mpt_grad_nonfinite(g16, n, inv_S, flag, stream=None):
    _check(lib().mpt_grad_nonfinite(_dptr(g16), n, float(inv_S), _dptr(flag), _stream_ptr(stream)))


def mpt_update_flat(g16, w32, v, w16, n, inv_S, lr, mu, use_momentum, detect, flags, stream=None):
    _check(lib().mpt_update_flat(_dptr(g16), _dptr(w32), _dptr(v), _dptr(w16), n, float(inv_S), float(lr), float(mu),
                                 int(bool(use_momentum)), int(bool(detect)), _dptr(flags), _stream_ptr(stream)))


CLIP_SCRATCH_BYTES = 16384


def mpt_update_flat_opt(opt, g16, w32, s1, s2, w16, n, inv_S, b1t, b2t, detect, flags, clip_scratch=None, stream=None):
    _check(lib().mpt_update_flat_opt(C.byref(opt), _dptr(g16), _dptr(w32), _dptr(s1), _dptr(s2), _dptr(w16), n,
                                     float(inv_S), float(b1t), float(b2t), int(bool(detect)), _dptr(flags),
                                     _dptr(clip_scratch), _stream_ptr(stream)))


def mpt_softmax_ce(z, ldz, labels, B, Cn, S, dz, lddz, row_loss, loss, bad_labels=None, stream=None, status=None):
    _check(lib().mpt_softmax_ce(_dptr(z), ldz, _dptr(labels), B, Cn, float(S), _dptr(dz), lddz, _dptr(row_loss),
                                _dptr(loss), _dptr(bad_labels), _dptr(status), _stream_ptr(stream)))


def mpt_softmax_ce_static(z, ldz, labels, B, Cn, S, dz, lddz, loss, bad_labels=None, stream=None, status=None):
    """mpt_softmax_ce for callers that cannot provide the float[B] scratch: the per-row losses
    live in a fixed array inside the library (B <= 65536; calls that overlap on the GPU race)."""
    _check(lib().mpt_softmax_ce_static(_dptr(z), ldz, _dptr(labels), B, Cn, float(S), _dptr(dz), lddz, _dptr(loss),
                                       _dptr(bad_labels), _dptr(status), _stream_ptr(stream)))


def mpt_sm_clock_probe(window_us, mhz, stream=None):
    """Enqueues the one-warp clock probe: mhz (a float32 CUDA tensor element) receives the SM clock in MHz."""
    _check(lib().mpt_sm_clock_probe(int(window_us), _dptr(mhz), _stream_ptr(stream)))


def mpt_selftest_wait_timeout(limit_us, status, stream=None) -> int:
    """Makes one bounded device-side wait run out on purpose; returns the library's code
    (MPT_ERR_TIMEOUT = -6 is the expected outcome) instead of raising."""
    return int(lib().mpt_selftest_wait_timeout(int(limit_us), _dptr(status), _stream_ptr(stream)))


def mpt_version() -> str:
    return lib().mpt_version().decode()


# ------------------------------------------------------------------ LSTM layer

def mpt_lstm_cell_forward(B, H, K, xr, ldxr, Wg, ldw, bias16, c_prev, ldcp, acts, ldacts, c_out, ldco, h_out, ldh, flags=0,
                          status=None, stream=None):
    _check(lib().mpt_lstm_cell_forward(B, H, K, _dptr(xr), ldxr, _dptr(Wg), ldw, _dptr(bias16), _dptr(c_prev), ldcp,
                                       _dptr(acts), ldacts, _dptr(c_out), ldco, _dptr(h_out), ldh, flags, _dptr(status),
                                       _stream_ptr(stream)))


def mpt_lstm_cell_backward(B, H, dh, lddh, dc_next, lddc, acts, ldacts, c_prev, ldcp, c16, ldc, dG, lddg, dc_prev, lddcp,
                           stream=None):
    _check(lib().mpt_lstm_cell_backward(B, H, _dptr(dh), lddh, _dptr(dc_next), lddc, _dptr(acts), ldacts, _dptr(c_prev), ldcp,
                                        _dptr(c16), ldc, _dptr(dG), lddg, _dptr(dc_prev), lddcp, _stream_ptr(stream)))


def mpt_bias_grad(dG, rows, cols, ld, parts, db16, nonfinite_flag=None, stream=None):
    _check(lib().mpt_bias_grad(_dptr(dG), rows, cols, ld, _dptr(parts), _dptr(db16), _dptr(nonfinite_flag), _stream_ptr(stream)))


def mpt_add_f16(a, lda, b, ldb, out, ldo, rows, cols, stream=None):
    _check(lib().mpt_add_f16(_dptr(a), lda, _dptr(b), ldb, _dptr(out), ldo, rows, cols, _stream_ptr(stream)))


class LstmLayer:
    """Device buffers of one LSTM layer with projection plus the two calls that run it.  Holds
    torch tensors (int16 views of FP16 bits) only to own the memory; all arithmetic happens in
    mpt_lstm_forward / mpt_lstm_backward."""

    def __init__(self, T, B, I, H, P):
        import torch
        self.desc = LstmDesc(T, B, I, H, P)
        z16 = lambda *shape: torch.zeros(shape, dtype=torch.int16, device="cuda")  # noqa: E731
        self.Wg16, self.bias16, self.Wp16 = z16(4 * H, I + P), z16(4 * H), z16(P, H)
        self.xr, self.c, self.h, self.acts = z16(T + 1, B, I + P), z16(T + 1, B, H), z16(T, B, H), z16(T, B, 4 * H)
        self.dr_ext, self.dxr, self.drtot, self.dG = z16(T, B, P), z16(T, B, I + P), z16(T, B, P), z16(T, B, 4 * H)
        self.dh, self.dc = z16(B, H), z16(2, B, H)
        self.dWg16, self.dWp16, self.dbias16 = z16(4 * H, I + P), z16(P, H), z16(4 * H)
        self.bias_parts = torch.zeros((8, 4 * H), dtype=torch.float32, device="cuda")
        self.status = torch.zeros(16, dtype=torch.int32, device="cuda")
        self.nonfinite_flag = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws_bytes = mpt_gemm_workspace_bytes(OP_FWD, B, P, H)
        self.splitk_ws = torch.zeros(max(ws_bytes, 16) // 4, dtype=torch.float32, device="cuda")
        self.tensors = LstmTensors(*([getattr(self, n if n != "status_dev" else "status").data_ptr() for n in _LSTM_FIELDS]
                                     + [self.splitk_ws.data_ptr() if ws_bytes else None, ws_bytes]))

    def forward(self, stream=None):
        _check(lib().mpt_lstm_forward(C.byref(self.desc), C.byref(self.tensors), _stream_ptr(stream)))

    def backward(self, stream=None):
        self.nonfinite_flag.zero_()
        _check(lib().mpt_lstm_backward(C.byref(self.desc), C.byref(self.tensors), _stream_ptr(stream)))

    def device_error(self) -> int:
        return int(self.status[3].item())


LSTM_T = dict(Wg32=0, Wp32=1, bias32=2, Wg16=3, Wp16=4, bias16=5, dWg16=6, dWp16=7, dbias16=8, s1_Wg32=9, s1_Wp32=10,
              s1_bias32=11, xr16=12, dr_ext16=13)


class LstmTrainer:
    """One mpt_lstm_ctx over a torch-allocated workspace: the LSTM layer with projection trained
    with loss scaling (mpt_lstm_train_step).  Argument marshalling only."""

    def __init__(self, T, B, I, H, P, S, optimizer, device="cuda:0", stream=None):
        import torch
        self.desc = LstmDesc(T, B, I, H, P)
        self.T, self.B, self.I, self.H, self.P = T, B, I, H, P
        self.optimizer = optimizer
        self.stream = stream
        out = C.c_size_t(0)
        _check(lib().mpt_lstm_workspace_bytes(C.byref(self.desc), C.byref(optimizer), C.byref(out)))
        nbytes = int(out.value)
        with torch.cuda.device(torch.device(device)):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            self._ctx = C.c_void_p()
            _check(lib().mpt_lstm_create(C.byref(self.desc), float(S), C.byref(optimizer), C.c_void_p(base), nbytes,
                                         _stream_ptr(stream), C.byref(self._ctx)))
        self.workspace_bytes = nbytes

    def _ck(self, code):
        if code != OK:
            raise MptError(code, lib().mpt_lstm_last_error(self._ctx).decode())

    def set_params(self, Wg, bias, Wp):
        Wg = np.ascontiguousarray(Wg, dtype=np.float32)
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        Wp = np.ascontiguousarray(Wp, dtype=np.float32)
        assert Wg.shape == (4 * self.H, self.I + self.P) and bias.shape == (4 * self.H,) and Wp.shape == (self.P, self.H)
        self._ck(lib().mpt_lstm_set_params(self._ctx, _hptr(Wg), _hptr(bias), _hptr(Wp)))

    def train_step(self, x_dev, labels_dev, want=True):
        """x_dev: FP16 bits [T, B, I]; labels_dev: int32 [T*B].  Returns (loss, overflow) when `want`."""
        if not want:
            self._ck(lib().mpt_lstm_train_step(self._ctx, _dptr(x_dev), _dptr(labels_dev), None, None))
            return None
        loss, flag = C.c_float(0.0), C.c_int(0)
        self._ck(lib().mpt_lstm_train_step(self._ctx, _dptr(x_dev), _dptr(labels_dev), C.byref(loss), C.byref(flag)))
        return float(loss.value), int(flag.value)

    def get_tensor(self, name):
        T, B, I, H, P = self.T, self.B, self.I, self.H, self.P
        K = I + P
        by_param = dict(Wg=(4 * H, K), Wp=(P, H), bias=(4 * H,))
        if name == "xr16":
            shape = (T + 1, B, K)
        elif name == "dr_ext16":
            shape = (T, B, P)
        else:
            shape = next(v for k, v in by_param.items() if k in name)
        dt = np.float32 if name.endswith("32") else np.uint16
        out = np.empty(shape, dtype=dt)
        self._ck(lib().mpt_lstm_get_tensor(self._ctx, LSTM_T[name], _hptr(out), out.nbytes))
        return out

    def set_dynamic_scale(self, enable, growth_interval=2000, min_scale=2.0 ** -100, max_scale=2.0 ** 120):
        self._ck(lib().mpt_lstm_set_dynamic_scale(self._ctx, int(bool(enable)), int(growth_interval), float(min_scale),
                                                  float(max_scale)))

    def get_scale(self):
        s = C.c_float(0.0)
        self._ck(lib().mpt_lstm_get_scale(self._ctx, C.byref(s)))
        return float(s.value)

    def close(self):
        if getattr(self, "_ctx", None):
            lib().mpt_lstm_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ------------------------------------------------------------------ data-parallel step

DP_MAX_REPLICAS = 16
DP_HANDLE_BYTES = 64


def mpt_dp_shard(n, R, rank):
    """Elements [lo, hi) of the flat parameter array that replica `rank` of R owns (host only)."""
    lo, hi = C.c_size_t(0), C.c_size_t(0)
    _check(lib().mpt_dp_shard(int(n), int(R), int(rank), C.byref(lo), C.byref(hi)))
    return int(lo.value), int(hi.value)


def _addr(x):
    """Device address of a tensor, a DeviceBuffer or a plain integer."""
    if isinstance(x, int):
        return x
    if isinstance(x, DeviceBuffer):
        return x.ptr
    return x.data_ptr()


def mpt_dp_step_flat(g16_peers, flag_peers, w16_peers, w32_shard, v_shard, n, R, rank, S, lr, mu, flags, stream=None):
    """One replica's part of the data-parallel step: the *_peers arguments are sequences of R device
    buffers (tensors, DeviceBuffers or addresses) in replica order, entry `rank` being this replica's."""
    assert len(g16_peers) == R and len(flag_peers) == R and len(w16_peers) == R
    tab = lambda xs: (C.c_void_p * R)(*[_addr(x) for x in xs])
    _check(lib().mpt_dp_step_flat(tab(g16_peers), tab(flag_peers), tab(w16_peers),
                                  None if w32_shard is None else C.c_void_p(_addr(w32_shard)),
                                  None if v_shard is None else C.c_void_p(_addr(v_shard)),
                                  int(n), int(R), int(rank), float(S), float(lr), float(mu), C.c_void_p(_addr(flags)),
                                  _stream_ptr(stream)))


DP_NORM_SCRATCH_BYTES = 8192


def mpt_dp_norm_flat(g16_peers, n, R, rank, S, scratch, norm_slot, stream=None):
    """First half of clipping in data-parallel mode: this replica's shard of the squared norm of the
    mean unscaled gradient, as a double in norm_slot (memory the other replicas can map)."""
    assert len(g16_peers) == R
    tab = (C.c_void_p * R)(*[_addr(x) for x in g16_peers])
    _check(lib().mpt_dp_norm_flat(tab, int(n), int(R), int(rank), float(S), C.c_void_p(_addr(scratch)),
                                  C.c_void_p(_addr(norm_slot)), _stream_ptr(stream)))


def mpt_dp_step_flat_opt(opt, g16_peers, flag_peers, w16_peers, w32_shard, s1_shard, s2_shard, n, R, rank, S, b1t, b2t,
                         flags, stream=None, norm_peers=None, clip_out=None):
    """mpt_dp_step_flat with any optimizer kind and weight decay; with opt.clip_norm > 0 also
    norm_peers (the R replicas' norm slots, after mpt_dp_norm_flat on every replica) and clip_out
    (two floats of this replica: coefficient, norm)."""
    assert len(g16_peers) == R and len(flag_peers) == R and len(w16_peers) == R
    tab = lambda xs: (C.c_void_p * R)(*[_addr(x) for x in xs])
    ptr = lambda x: None if x is None else C.c_void_p(_addr(x))
    _check(lib().mpt_dp_step_flat_opt(C.byref(opt), tab(g16_peers), tab(flag_peers), tab(w16_peers), ptr(w32_shard),
                                      ptr(s1_shard), ptr(s2_shard), int(n), int(R), int(rank), float(S), float(b1t), float(b2t),
                                      C.c_void_p(_addr(flags)), None if norm_peers is None else tab(norm_peers), ptr(clip_out),
                                      _stream_ptr(stream)))


class DeviceBuffer:
    """Device memory that other processes can map: either this process's own allocation (made by
    the library from the driver's allocator) or a mapping of a peer's, opened from its handle.
    `tensor(dtype)` views it as a torch tensor without copying."""

    def __init__(self, nbytes=None, handle=None):
        p = C.c_void_p(0)
        if handle is None:
            _check(lib().mpt_dp_alloc(int(nbytes), C.byref(p)))
            self.owned = True
        else:
            assert len(handle) == DP_HANDLE_BYTES
            buf = (C.c_uint8 * DP_HANDLE_BYTES).from_buffer_copy(handle)
            _check(lib().mpt_dp_open(buf, C.byref(p)))
            self.owned = False
        self.ptr = int(p.value)
        self.nbytes = nbytes

    def export(self) -> bytes:
        assert self.owned
        buf = (C.c_uint8 * DP_HANDLE_BYTES)()
        _check(lib().mpt_dp_export(C.c_void_p(self.ptr), buf))
        return bytes(buf)

    def tensor(self, dtype, count=None):
        import torch
        item = torch.empty((), dtype=dtype).element_size()
        n = self.nbytes // item if count is None else int(count)
        typestr = {torch.uint8: "|u1", torch.int16: "<i2", torch.float16: "<f2", torch.float32: "<f4",
                   torch.int32: "<i4", torch.uint16: "<u2"}[dtype]

        class _View:
            __cuda_array_interface__ = dict(shape=(n,), typestr=typestr, data=(self.ptr, False), version=2)

        return torch.as_tensor(_View(), device="cuda")

    def close(self):
        if self.ptr:
            if self.owned:
                _check(lib().mpt_dp_free(C.c_void_p(self.ptr)))
            else:
                _check(lib().mpt_dp_close(C.c_void_p(self.ptr)))
            self.ptr = 0


def dp_exchange_handles(handles: dict, group=None):
    """All-gather of each replica's {name: handle bytes} through torch.distributed (any backend):
    returns a list over replicas of such dicts, in rank order."""
    import torch.distributed as dist
    out = [None] * dist.get_world_size(group)
    dist.all_gather_object(out, handles, group=group)
    return out


class DataParallelFlat:
    """Replica `rank` of R for a flat parameter array of n elements: owns the exchange buffers
    (scaled FP16 gradient, FP16 weights, overflow words), maps the peers' buffers, holds the FP32
    master and momentum of its own shard only, and runs the one-kernel step.  Replicas are
    processes of a torch.distributed group (one per GPU); the group's barrier orders them around
    the step (host-synchronous: the stream is drained first)."""

    def __init__(self, n, S, lr, mu, group=None):
        import torch
        import torch.distributed as dist
        self.group = group
        self.R, self.rank = dist.get_world_size(group), dist.get_rank(group)
        self.n, self.S, self.lr, self.mu = int(n), float(S), float(lr), float(mu)
        self.lo, self.hi = mpt_dp_shard(n, self.R, self.rank)
        pad = (self.n + 7) // 8 * 16
        self._own = dict(g16=DeviceBuffer(pad), w16=DeviceBuffer(pad), flags=DeviceBuffer(256))
        self.g16 = self._own["g16"].tensor(torch.int16, self.n)
        self.w16 = self._own["w16"].tensor(torch.int16, self.n)
        self.flags = self._own["flags"].tensor(torch.int32, 2)
        self.flags.zero_()
        cnt = max(self.hi - self.lo, 1)
        self.w32 = torch.zeros(cnt, dtype=torch.float32, device="cuda")
        self.v = torch.zeros(cnt, dtype=torch.float32, device="cuda") if self.mu != 0.0 else None
        table = dp_exchange_handles({k: b.export() for k, b in self._own.items()}, group)
        self._peers = []
        for q in range(self.R):
            self._peers.append(self._own if q == self.rank else {k: DeviceBuffer(handle=h) for k, h in table[q].items()})

    def _barrier(self):
        import torch
        import torch.distributed as dist
        torch.cuda.current_stream().synchronize()
        dist.barrier(group=self.group)

    def step(self):
        """Gradients (self.g16) and overflow word (self.flags[0]) of every replica must have been
        produced on the current stream.  Returns True when the step was skipped everywhere."""
        self._barrier()
        mpt_dp_step_flat([p["g16"] for p in self._peers], [p["flags"] for p in self._peers],
                         [p["w16"] for p in self._peers], self.w32, self.v, self.n, self.R, self.rank, self.S,
                         self.lr, self.mu, self._own["flags"])
        self._barrier()
        # every replica's kernel has finished: nobody reads this word again before the next step's
        # first barrier, which also drains the stream the clear is queued on
        skipped = bool(int(self.flags[0].item()) != 0)
        self.flags.zero_()
        return skipped

    def close(self):
        self._barrier()
        for q, p in enumerate(self._peers):
            if q != self.rank:
                for b in p.values():
                    b.close()
        self._barrier()
        for b in self._own.values():
            b.close()


class DataParallelMLP:
    """Replica `rank` of R of an MLP context in a torch.distributed group (one process per GPU):
    the context's workspace is shareable, the replicas map each other's workspaces, and step() runs
    the one-kernel data-parallel step between two barriers.  Every replica feeds its own part of
    the batch (equal sizes) through forward() / backward_scaled() of `ctx`."""

    def __init__(self, layers, S, lr, momentum=0.0, max_batch=1, group=None, optimizer=None, shard_state=False,
                 overlap=False):
        """shard_state: keep FP32 master and optimizer state for this replica's shard only (mpt_create_dp).
        overlap: pull and add the replicas' gradients layer by layer beside the backward pass (interprocess
        events; call ctx.backward_scaled(labels, want_loss=False) so that the pass is only enqueued)."""
        import torch.distributed as dist
        self.group = group
        self.R, self.rank = dist.get_world_size(group), dist.get_rank(group)
        self.ctx = Context(layers, S, lr, momentum, max_batch, shareable=True, optimizer=optimizer,
                           shard=(self.R, self.rank) if shard_state and self.R > 1 else None)
        lay = self.ctx.dp_layout()
        own = self.ctx.workspace
        table = dp_exchange_handles({"ws": own.export(), "skew": self.ctx._ws_ptr - own.ptr}, group)
        self._maps = []
        g, f, w = [], [], []
        for q in range(self.R):
            if q == self.rank:
                base = self.ctx._ws_ptr
            else:
                m = DeviceBuffer(handle=table[q]["ws"])
                self._maps.append(m)
                base = m.ptr + table[q]["skew"]
            g.append(base + lay.g16_offset)
            w.append(base + lay.w16_offset)
            f.append(base + lay.flags_offset)
        if self.R > 1:
            self.ctx.dp_attach(self.R, self.rank, g, f, w)
        self.overlap = bool(overlap) and self.R > 1
        if self.overlap:
            mine = self.ctx.dp_overlap_events()
            handles = [None] * self.R
            dist.all_gather_object(handles, mine, group=group)
            self.ctx.dp_overlap_attach(handles, self.rank)
        self.shard = mpt_dp_shard(lay.n, self.R, self.rank)

    def _barrier(self):
        import torch
        import torch.distributed as dist
        torch.cuda.current_stream().synchronize()
        dist.barrier(group=self.group)

    def step(self):
        """All replicas call this after their backward_scaled(); returns True if the step was skipped."""
        if self.overlap:
            import torch.distributed as dist
            dist.barrier(group=self.group)      # every replica has ENQUEUED its backward pass; nobody waits for a GPU here
            self.ctx.dp_reduce_async()
            if self.ctx.optimizer.clip_norm > 0.0:
                dist.barrier(group=self.group)  # every replica has enqueued the publication of its part of the norm
            overflow = self.ctx.step()          # waits on the streams for the sums and for every replica's pass
            self._barrier()
            return bool(overflow)
        self._barrier()
        if self.R > 1 and self.ctx.optimizer.clip_norm > 0.0:
            self.ctx.dp_norm()          # every replica's part of the norm, then all of them visible to all
            self._barrier()
        overflow = self.ctx.step()
        self._barrier()
        return bool(overflow)

    def close(self):
        self._barrier()
        for m in self._maps:
            m.close()
        self._maps = []
        self._barrier()
        self.ctx.close()
