"""ctypes access to the CPU oracle (mpo.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this module, and this module never imports them.

The shared object is compiled on first use with gcc (see ``build``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mpo.c")
_LIB = os.path.join(_HERE, "libmpo.so")

OP_FWD, OP_DGRAD, OP_WGRAD = 0, 1, 2

_lib = None


def build(force: bool = False) -> str:
    """Compile mpo.c into libmpo.so (gcc, separately rounded binary32 ops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        c = ctypes
        L.mpo_h2f.restype = c.c_float
        L.mpo_h2f.argtypes = [c.c_uint16]
        L.mpo_f2h.restype = c.c_uint16
        L.mpo_f2h.argtypes = [c.c_float]
        L.mpo_h2f_array.restype = None
        L.mpo_h2f_array.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t]
        L.mpo_f2h_array.restype = None
        L.mpo_f2h_array.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t]
        L.mpo_f2h_bits_range.restype = None
        L.mpo_f2h_bits_range.argtypes = [c.c_uint32, c.c_uint32, c.c_void_p]
        L.mpo_num_threads.restype = c.c_int
        L.mpo_num_threads.argtypes = []
        L.mpo_gemm_f16.restype = None
        L.mpo_gemm_f16.argtypes = [c.c_int, c.c_int, c.c_int, c.c_int,
                                   c.c_void_p, c.c_int, c.c_void_p, c.c_int,
                                   c.c_void_p, c.c_int, c.c_int,
                                   c.c_void_p, c.c_int, c.c_void_p, c.c_void_p,
                                   c.c_int, c.c_int]
        L.mpo_gemm_f16_element.restype = c.c_uint16
        L.mpo_gemm_f16_element.argtypes = [c.c_int, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int,
                                           c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p]
        L.mpo_softmax_ce.restype = c.c_int
        L.mpo_softmax_ce.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_int, c.c_float,
                                     c.c_void_p, c.c_int, c.c_void_p, c.c_void_p]
        L.mpo_grad_nonfinite.restype = c.c_int
        L.mpo_grad_nonfinite.argtypes = [c.c_void_p, c.c_size_t, c.c_float]
        L.mpo_update_apply.restype = None
        L.mpo_update_apply.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t,
                                       c.c_float, c.c_float, c.c_float, c.c_int]
        L.mpo_update_apply_opt.restype = None
        L.mpo_update_apply_opt.argtypes = [c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                           c.c_size_t] + [c.c_float] * 8
        L.mpo_grad_sqnorm.restype = c.c_double
        L.mpo_grad_sqnorm.argtypes = [c.c_void_p, c.c_size_t, c.c_float]
        L.mpo_update_apply_clip.restype = None
        L.mpo_update_apply_clip.argtypes = [c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                            c.c_size_t] + [c.c_float] * 9
        L.mpo_lstm_cell_fwd.restype = None
        L.mpo_lstm_cell_fwd.argtypes = [c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_void_p,
                                        c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int,
                                        c.c_void_p, c.c_void_p]
        L.mpo_lstm_cell_bwd.restype = None
        L.mpo_lstm_cell_bwd.argtypes = [c.c_int, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int,
                                        c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int]
        L.mpo_bias_grad.restype = None
        L.mpo_bias_grad.argtypes = [c.c_void_p, c.c_size_t, c.c_int, c.c_int, c.c_void_p, c.c_void_p]
        L.mpo_add_f16.restype = None
        L.mpo_add_f16.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_int, c.c_int]
        L.mpo_dp_update_apply_opt.restype = None
        L.mpo_dp_update_apply_opt.argtypes = [c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                              c.c_size_t, c.c_float, c.c_float, c.c_float, c.c_float, c.c_float, c.c_float,
                                              c.c_float, c.c_float]
        L.mpo_dp_grad_sqnorm.restype = c.c_double
        L.mpo_dp_grad_sqnorm.argtypes = [c.c_void_p, c.c_int, c.c_size_t, c.c_float]
        L.mpo_dp_update_apply_clip.restype = None
        L.mpo_dp_update_apply_clip.argtypes = [c.c_int, c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                               c.c_size_t, c.c_float, c.c_float, c.c_float, c.c_float, c.c_float, c.c_float,
                                               c.c_float, c.c_float, c.c_float]
        L.mpo_dp_update_apply.restype = None
        L.mpo_dp_update_apply.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t,
                                          c.c_float, c.c_float, c.c_float, c.c_int]
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().mpo_num_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a) -> np.ndarray:
    """View/convert an array of binary16 values as contiguous uint16 bit patterns."""
    a = np.asarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("expected float16 or uint16 bit patterns, got %s" % a.dtype)
    return a


def h2f(h) -> np.ndarray:
    h = np.ascontiguousarray(_u16(h))
    out = np.empty(h.shape, dtype=np.float32)
    lib().mpo_h2f_array(_ptr(h), _ptr(out), h.size)
    return out


def f2h(f) -> np.ndarray:
    """binary32 -> binary16 bit patterns (uint16), round to nearest even."""
    f = np.ascontiguousarray(np.asarray(f, dtype=np.float32))
    out = np.empty(f.shape, dtype=np.uint16)
    lib().mpo_f2h_array(_ptr(f), _ptr(out), f.size)
    return out


def f2h_bits_range(first: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.uint16)
    lib().mpo_f2h_bits_range(first, count, _ptr(out))
    return out


def gemm_f16(op, A, B, relu=False, mask=None, want_exact=False, rows=None):
    """Linear-layer product in the mixed-precision recipe (paper section 3.3).

    op 0: C[M,N] = A[M,K] . B[N,K]^T ; op 1: C[M,N] = A[M,K] . B[K,N] ;
    op 2: C[M,N] = A[K,M]^T . B[K,N].  A, B, mask: 2-D uint16/float16 arrays (row
    strides may exceed the row length).  Returns uint16 bit patterns, plus
    (exact, absdot) float64 arrays when want_exact.
    """
    A = _u16(A)
    B = _u16(B)
    assert A.ndim == 2 and B.ndim == 2
    assert A.strides[1] == 2 and B.strides[1] == 2
    if op == OP_FWD:
        M, K = A.shape
        N, K2 = B.shape
    elif op == OP_DGRAD:
        M, K = A.shape
        K2, N = B.shape
    elif op == OP_WGRAD:
        K, M = A.shape
        K2, N = B.shape
    else:
        raise ValueError("op")
    assert K == K2, (A.shape, B.shape, op)
    lda = A.strides[0] // 2 if A.shape[0] > 1 else A.shape[1]
    ldb = B.strides[0] // 2 if B.shape[0] > 1 else B.shape[1]
    C = np.zeros((M, N), dtype=np.uint16)
    ex = np.zeros((M, N), dtype=np.float64) if want_exact else None
    ab = np.zeros((M, N), dtype=np.float64) if want_exact else None
    mk = None
    ldm = 0
    if mask is not None:
        mk = _u16(mask)
        assert mk.shape == (M, N) and mk.strides[1] == 2
        ldm = mk.strides[0] // 2 if M > 1 else N
    r0, r1 = (0, M) if rows is None else rows
    lib().mpo_gemm_f16(op, M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), N, int(bool(relu)),
                       _ptr(mk), ldm, _ptr(ex), _ptr(ab), r0, r1)
    if want_exact:
        return C, ex, ab
    return C


def gemm_f16_element(op, A, B, m, n, relu=False):
    """One output element (rounded bits, exact double sum, sum of |products|)."""
    A = _u16(A)
    B = _u16(B)
    K = A.shape[0] if op == OP_WGRAD else A.shape[1]
    lda = A.strides[0] // 2
    ldb = B.strides[0] // 2
    ex = ctypes.c_double(0.0)
    ab = ctypes.c_double(0.0)
    h = lib().mpo_gemm_f16_element(op, K, _ptr(A), lda, _ptr(B), ldb, int(m), int(n), int(bool(relu)),
                                   ctypes.byref(ex), ctypes.byref(ab))
    return int(h), ex.value, ab.value


def softmax_ce(z, labels, S):
    """Softmax cross-entropy forward + scaled backward (paper sections 3.2, 3.3).

    Returns (dz uint16 [B,C], row_loss float32 [B], mean loss float, n_bad_labels).
    """
    z = _u16(z)
    assert z.ndim == 2 and z.strides[1] == 2
    Bn, C = z.shape
    ldz = z.strides[0] // 2 if Bn > 1 else C
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    dz = np.zeros((Bn, C), dtype=np.uint16)
    rl = np.zeros(Bn, dtype=np.float32)
    loss = ctypes.c_float(0.0)
    bad = lib().mpo_softmax_ce(_ptr(z), ldz, _ptr(labels), Bn, C, float(S), _ptr(dz), C, _ptr(rl),
                               ctypes.byref(loss))
    return dz, rl, float(loss.value), int(bad)


def grad_nonfinite(g16, inv_S) -> int:
    g = np.ascontiguousarray(_u16(g16)).reshape(-1)
    return int(lib().mpo_grad_nonfinite(_ptr(g), g.size, float(inv_S)))


def update_apply(g16, w32, v, w16, inv_S, lr, mu, use_momentum) -> None:
    """In-place master update on contiguous arrays (caller has checked the flag)."""
    g = _u16(g16)
    for a in (g, w32, w16) + ((v,) if v is not None else ()):
        assert a.flags["C_CONTIGUOUS"]
    assert w32.dtype == np.float32 and w16.dtype == np.uint16
    if use_momentum:
        assert v is not None and v.dtype == np.float32
    lib().mpo_update_apply(_ptr(g), _ptr(w32), _ptr(v) if use_momentum else None, _ptr(w16), g.size,
                           float(inv_S), float(lr), float(mu), int(bool(use_momentum)))


OPT_SGD, OPT_NESTEROV, OPT_ADAGRAD, OPT_ADAM = 0, 1, 2, 3


def update_apply_opt(kind, g16, w32, s1, s2, w16, inv_S, lr, mu, b2=0.0, eps=0.0, wd=0.0, bc1=1.0, bc2=1.0) -> None:
    """In-place optimizer step of the given kind on contiguous arrays (see mpo.c for the op order)."""
    g = _u16(g16)
    for a in (g, w32, w16, s1, s2):
        if a is not None:
            assert a.flags["C_CONTIGUOUS"]
    lib().mpo_update_apply_opt(int(kind), _ptr(g), _ptr(w32), _ptr(s1), _ptr(s2), _ptr(w16), g.size, float(inv_S),
                               float(lr), float(mu), float(b2), float(eps), float(wd), float(bc1), float(bc2))


def grad_sqnorm(g16, inv_S) -> float:
    """Sum of squares of the unscaled gradients, accumulated in double."""
    g = np.ascontiguousarray(_u16(g16)).reshape(-1)
    return float(lib().mpo_grad_sqnorm(_ptr(g), g.size, float(inv_S)))


def clip_coef(total_sq, clip_norm) -> np.float32:
    """coef = min(1, clip / (sqrt(total) + 1e-6)), rounded to binary32.  The bound is a binary32
    parameter of the optimizer: the quotient is formed in double from its binary32 value."""
    return np.float32(min(1.0, float(np.float32(clip_norm)) / (float(np.sqrt(total_sq)) + 1e-6)))


def update_apply_clip(kind, g16, w32, s1, s2, w16, inv_S, coef, lr, mu, b2=0.0, eps=0.0, wd=0.0, bc1=1.0, bc2=1.0) -> None:
    g = _u16(g16)
    lib().mpo_update_apply_clip(int(kind), _ptr(g), _ptr(w32), _ptr(s1), _ptr(s2), _ptr(w16), g.size, float(inv_S),
                                float(coef), float(lr), float(mu), float(b2), float(eps), float(wd), float(bc1), float(bc2))


def _ld(a):
    """Row pitch in elements of a 2-D array whose rows are contiguous."""
    assert a.ndim == 2 and a.strides[1] == a.itemsize
    return a.strides[0] // a.itemsize if a.shape[0] > 1 else a.shape[1]


def lstm_cell_fwd(xr, Wg, bias16, c_prev, want_pre=False):
    """One time step of the LSTM cell (see mpo.c): xr [B,K], Wg [4H,K] gate-interleaved rows,
    bias16 [4H], c_prev [B,H].  Returns (acts [B,4H], c [B,H], h [B,H]) as uint16 bit patterns,
    plus (pre32 float32 [B,4H], absdot float64 [B,4H]) when want_pre."""
    xr, Wg, bias16, c_prev = _u16(xr), _u16(Wg), np.ascontiguousarray(_u16(bias16)), _u16(c_prev)
    B, K = xr.shape
    N = Wg.shape[0]
    H = N // 4
    assert N == 4 * H and Wg.shape[1] == K and c_prev.shape == (B, H) and bias16.shape == (N,)
    acts = np.zeros((B, N), dtype=np.uint16)
    c = np.zeros((B, H), dtype=np.uint16)
    h = np.zeros((B, H), dtype=np.uint16)
    pre = np.zeros((B, N), dtype=np.float32) if want_pre else None
    ab = np.zeros((B, N), dtype=np.float64) if want_pre else None
    lib().mpo_lstm_cell_fwd(B, H, K, _ptr(xr), _ld(xr), _ptr(Wg), _ld(Wg), _ptr(bias16), _ptr(c_prev), _ld(c_prev),
                            _ptr(acts), N, _ptr(c), H, _ptr(h), H, _ptr(pre), _ptr(ab))
    if want_pre:
        return acts, c, h, pre, ab
    return acts, c, h


def lstm_cell_bwd(dh, dc_next, acts, c_prev, c):
    """Backward of the gate arithmetic of one time step: returns (dG [B,4H], dc_prev [B,H])."""
    dh, acts, c_prev, c = _u16(dh), _u16(acts), _u16(c_prev), _u16(c)
    B, H = dh.shape
    dcn = None if dc_next is None else _u16(dc_next)
    dG = np.zeros((B, 4 * H), dtype=np.uint16)
    dcp = np.zeros((B, H), dtype=np.uint16)
    lib().mpo_lstm_cell_bwd(B, H, _ptr(dh), _ld(dh), _ptr(dcn), _ld(dcn) if dcn is not None else 0, _ptr(acts), _ld(acts),
                            _ptr(c_prev), _ld(c_prev), _ptr(c), _ld(c), _ptr(dG), 4 * H, _ptr(dcp), H)
    return dG, dcp


def bias_grad(dG):
    """Column sums (binary32, ascending rows) of a [rows, cols] FP16 array: (db16, db32)."""
    dG = _u16(dG)
    rows, cols = dG.shape
    db16 = np.zeros(cols, dtype=np.uint16)
    db32 = np.zeros(cols, dtype=np.float32)
    lib().mpo_bias_grad(_ptr(dG), rows, cols, _ld(dG), _ptr(db16), _ptr(db32))
    return db16, db32


def add_f16(a, b):
    a, b = _u16(a), _u16(b)
    out = np.zeros(a.shape, dtype=np.uint16)
    lib().mpo_add_f16(_ptr(a), _ld(a), _ptr(b), _ld(b), _ptr(out), a.shape[1], a.shape[0], a.shape[1])
    return out


def dp_inv_scale(S, R) -> np.float32:
    """1 / (S * R) in binary32: one multiplication, one division."""
    return np.float32(1.0) / (np.float32(S) * np.float32(R))


def dp_update_apply(g16_list, w32, v, w16, S, lr, mu, use_momentum) -> None:
    """In-place data-parallel master update (see mpo.c): g16_list holds one contiguous gradient
    array per replica, in replica order.  The caller has checked every replica's overflow flag."""
    gs = [np.ascontiguousarray(_u16(g)).reshape(-1) for g in g16_list]
    R = len(gs)
    assert R >= 1 and all(g.size == gs[0].size for g in gs)
    for a in (w32, w16) + ((v,) if v is not None else ()):
        assert a.flags["C_CONTIGUOUS"]
    assert w32.dtype == np.float32 and w16.dtype == np.uint16 and w32.size == gs[0].size
    table = (ctypes.c_void_p * R)(*[g.ctypes.data for g in gs])
    lib().mpo_dp_update_apply(table, R, _ptr(w32), _ptr(v) if use_momentum else None, _ptr(w16), gs[0].size,
                              float(dp_inv_scale(S, R)), float(lr), float(mu), int(bool(use_momentum)))


def dp_grad_sqnorm(g16_list, S) -> float:
    """Sum of squares (double) of the mean unscaled gradient of the replicas (see mpo.c)."""
    gs = [np.ascontiguousarray(_u16(g)).reshape(-1) for g in g16_list]
    R = len(gs)
    table = (ctypes.c_void_p * R)(*[g.ctypes.data for g in gs])
    return float(lib().mpo_dp_grad_sqnorm(table, R, gs[0].size, float(dp_inv_scale(S, R))))


def dp_update_apply_clip(kind, g16_list, w32, s1, s2, w16, S, coef, lr, mu, b2=0.0, eps=0.0, wd=0.0, bc1=1.0, bc2=1.0) -> None:
    """dp_update_apply_opt with the clipping coefficient applied to the mean gradient."""
    gs = [np.ascontiguousarray(_u16(g)).reshape(-1) for g in g16_list]
    R = len(gs)
    assert R >= 1 and all(g.size == gs[0].size for g in gs)
    table = (ctypes.c_void_p * R)(*[g.ctypes.data for g in gs])
    lib().mpo_dp_update_apply_clip(int(kind), table, R, _ptr(w32), _ptr(s1), _ptr(s2), _ptr(w16), gs[0].size,
                                   float(dp_inv_scale(S, R)), float(coef), float(lr), float(mu), float(b2), float(eps),
                                   float(wd), float(bc1), float(bc2))


def dp_update_apply_opt(kind, g16_list, w32, s1, s2, w16, S, lr, mu, b2=0.0, eps=0.0, wd=0.0, bc1=1.0, bc2=1.0) -> None:
    """Data-parallel step with any optimizer kind (see mpo.c): mean of the replicas' gradients, then
    the op order of update_apply_opt."""
    gs = [np.ascontiguousarray(_u16(g)).reshape(-1) for g in g16_list]
    R = len(gs)
    assert R >= 1 and all(g.size == gs[0].size for g in gs)
    table = (ctypes.c_void_p * R)(*[g.ctypes.data for g in gs])
    lib().mpo_dp_update_apply_opt(int(kind), table, R, _ptr(w32), _ptr(s1), _ptr(s2), _ptr(w16), gs[0].size,
                                  float(dp_inv_scale(S, R)), float(lr), float(mu), float(b2), float(eps), float(wd),
                                  float(bc1), float(bc2))
