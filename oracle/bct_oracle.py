"""ctypes front end of the double-precision CPU oracle (TEST INFRASTRUCTURE).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this module; nothing in the CUDA product path does.  All arithmetic lives in
``bct_oracle.c``; this file builds it with gcc, marshals numpy arrays and moves
the caller's ``[B, T, H, d]`` layouts to the oracle's unit-major layout.

Semantics per (sequence, kv-head) unit and token (Method steps 2-5, Algorithm 1,
Illustration step 3 of the paper; read path = softmax attention over the
resident slots):

    read :  o_g  = softmax(read_scale * q_g . MK^T) . MV_{t-1}
    write:  MV_t = MV_{t-1} + softmax(write_scale * k_t . MK^T)^T . v_t

with a hard-append fill phase while fewer than ``capacity`` slots are resident.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

SKIP_FIRST_WRITE = 1
WRITE_THEN_READ = 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bct_oracle.c")
_LIB = os.path.join(_HERE, "libbct_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``bct_oracle.c`` into ``libbct_oracle.so`` next to it (gcc, OpenMP)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp%d" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                   "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        try:
            lib = ctypes.CDLL(_LIB)
        except OSError:
            build(force=True)
            lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        lib.bct_oracle_stream.restype = ctypes.c_int
        lib.bct_oracle_stream.argtypes = [
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
            ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
            dp, dp, dp, dp, dp, dp, ctypes.c_double, ctypes.c_double, ctypes.c_uint, ctypes.c_int]
        lib.bct_oracle_stream_eta.restype = ctypes.c_int
        lib.bct_oracle_stream_eta.argtypes = [
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
            ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
            dp, dp, dp, dp, dp, dp, dp, ctypes.c_double, ctypes.c_double, ctypes.c_uint, ctypes.c_int]
        lib.bct_oracle_stream_eps.restype = ctypes.c_int
        lib.bct_oracle_stream_eps.argtypes = [
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
            ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
            dp, dp, dp, dp, dp, dp, dp, ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_uint, ctypes.c_int]
        lib.bct_oracle_update_kv_backward.restype = ctypes.c_int
        lib.bct_oracle_update_kv_backward.argtypes = [
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int64, dp, dp, dp, dp, dp, ctypes.c_double,
            ctypes.c_double, dp, dp, dp, dp, ctypes.c_int]
        lib.bct_oracle_project.restype = ctypes.c_int
        lib.bct_oracle_project.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, dp, dp, dp, ctypes.c_int]
        lib.bct_oracle_write_weights.restype = ctypes.c_int
        lib.bct_oracle_write_weights.argtypes = [ctypes.c_int64, ctypes.c_int, dp, dp,
                                                 ctypes.c_double, dp]
        lib.bct_oracle_read_weights.restype = ctypes.c_int
        lib.bct_oracle_read_weights.argtypes = [ctypes.c_int64, ctypes.c_int, dp, dp,
                                                ctypes.c_double, dp]
        _lib = lib
    return _lib


def _dptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def write_weights(MK, wq, write_scale: float = 1.0) -> np.ndarray:
    """ww = softmax(write_scale * wq . MK^T) for one unit (Algorithm 1)."""
    MK = _f64(MK)
    wq = _f64(wq)
    C, d = MK.shape
    ww = np.empty(C, dtype=np.float64)
    rc = _load().bct_oracle_write_weights(C, d, _dptr(MK), _dptr(wq), float(write_scale), _dptr(ww))
    if rc != 0:
        raise RuntimeError("bct_oracle_write_weights failed")
    return ww


def read_weights(MK, q, read_scale: float) -> np.ndarray:
    """p = softmax(read_scale * q . MK^T) for one head over the rows of MK given."""
    MK = _f64(MK)
    q = _f64(q)
    n, d = MK.shape
    p = np.empty(n, dtype=np.float64)
    rc = _load().bct_oracle_read_weights(n, d, _dptr(MK), _dptr(q), float(read_scale), _dptr(p))
    if rc != 0:
        raise RuntimeError("bct_oracle_read_weights failed")
    return p


def project(x, W, nthreads: int = 0) -> np.ndarray:
    """y = x . W^T: x ``[..., K]`` (one row per token), W ``[N, K]`` (one row per output feature)
    -> ``[..., N]`` float64 (Algorithm 1: wq_t = W_wq x_t, wv_t = W_wv x_t)."""
    x = _f64(x)
    W = _f64(W)
    K = x.shape[-1]
    N = W.shape[0]
    assert W.shape == (N, K), (W.shape, K)
    x2 = np.ascontiguousarray(x.reshape(-1, K))
    y = np.empty((x2.shape[0], N), dtype=np.float64)
    rc = _load().bct_oracle_project(x2.shape[0], K, N, _dptr(x2), _dptr(W), _dptr(y), int(nthreads))
    if rc < 0:
        raise RuntimeError("bct_oracle_project failed")
    return y.reshape(x.shape[:-1] + (N,))


def round_bf16(a) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned as float64: the storage type of the
    step vectors when the cache is bfloat16."""
    f = np.ascontiguousarray(np.asarray(a, dtype=np.float32))
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


def layer_step_inputs(x, Wq, Wwq, Wwv, n_q_heads, n_kv_heads, head_dim, bf16: bool = True):
    """Projections of a block of tokens x ``[B, T, d_model]`` into the step vectors of the layer:
    q ``[B, T, Hq, d]``, k (= wq) and v (= wv) ``[B, T, Hkv, d]``, rounded to the step-vector
    storage type."""
    B, T = x.shape[0], x.shape[1]
    rnd = round_bf16 if bf16 else (lambda z: np.asarray(z, dtype=np.float32).astype(np.float64))
    q = rnd(project(x, Wq)).reshape(B, T, n_q_heads, head_dim)
    k = rnd(project(x, Wwq)).reshape(B, T, n_kv_heads, head_dim)
    v = rnd(project(x, Wwv)).reshape(B, T, n_kv_heads, head_dim)
    return q, k, v


def update_kv_backward(MK, wq, wv, dMV, eta=None, write_scale: float = 1.0, write_eps: float = 0.0, nthreads: int = 0):
    """Backward of Algorithm 1's UpdateKV (token-parallel form): MK ``[B, Hkv, C, d]`` (full cache), wq, wv
    ``[B, T, Hkv, d]``, eta ``[B, T, Hkv]`` or None, dMV = dL/dMV_N ``[B, Hkv, C, d]``.  Returns
    (dwq, dwv ``[B, T, Hkv, d]``, dMK ``[B, Hkv, C, d]``, deta ``[B, T, Hkv]``); dL/dMV_0 is dMV itself."""
    MK, wq, wv, dMV = _f64(MK), _f64(wq), _f64(wv), _f64(dMV)
    B, Hkv, C, d = MK.shape
    T = wq.shape[1]
    assert wq.shape == (B, T, Hkv, d) and wv.shape == (B, T, Hkv, d) and dMV.shape == (B, Hkv, C, d)
    U = B * Hkv
    qu = np.ascontiguousarray(wq.transpose(0, 2, 1, 3)).reshape(U, T, d)
    vu = np.ascontiguousarray(wv.transpose(0, 2, 1, 3)).reshape(U, T, d)
    eu = None
    if eta is not None:
        eta = _f64(eta)
        assert eta.shape == (B, T, Hkv), eta.shape
        eu = np.ascontiguousarray(eta.transpose(0, 2, 1)).reshape(U, T)
    dq, dv = np.empty((U, T, d)), np.empty((U, T, d))
    dmk, de = np.empty((U, C, d)), np.empty((U, T))
    rc = _load().bct_oracle_update_kv_backward(
        U, T, d, C, _dptr(MK.reshape(U, C, d)), _dptr(qu), _dptr(vu), _dptr(eu) if eu is not None else None,
        _dptr(dMV.reshape(U, C, d)), float(write_scale), float(write_eps), _dptr(dq), _dptr(dv), _dptr(dmk), _dptr(de),
        int(nthreads))
    if rc < 0:
        raise RuntimeError("bct_oracle_update_kv_backward failed")
    back = lambda a: np.ascontiguousarray(a.reshape(B, Hkv, T, d).transpose(0, 2, 1, 3))
    return back(dq), back(dv), dmk.reshape(B, Hkv, C, d), np.ascontiguousarray(de.reshape(B, Hkv, T).transpose(0, 2, 1))


class OracleCache:
    """Bounded cache of ``capacity`` slots for ``batch * n_kv_heads`` independent units.

    ``mk_init`` / ``mv_init``: ``[batch, n_kv_heads, init_len, head_dim]`` (the paper's
    MK and MV_0; ``mv_init=None`` with ``init_len > 0`` means zeros, one of the two
    initialisations the Method section allows).  ``read_scale=None`` means
    ``1/sqrt(head_dim)``; ``write_scale=None`` means 1.0 (Algorithm 1 prints no scale).
    ``write_eps``: slots whose write weight is below it keep their row (0 = the printed rule).
    """

    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, capacity, *, read_scale=None,
                 write_scale=None, init_len=0, mk_init=None, mv_init=None, flags=0,
                 nthreads=0, write_eps=0.0):
        if n_q_heads % n_kv_heads:
            raise ValueError("n_q_heads must be a multiple of n_kv_heads")
        if not (0 <= init_len <= capacity):
            raise ValueError("init_len out of range")
        self.B, self.Hq, self.Hkv, self.d, self.C = batch, n_q_heads, n_kv_heads, head_dim, capacity
        self.G = n_q_heads // n_kv_heads
        self.U = batch * n_kv_heads
        self.read_scale = float(1.0 / np.sqrt(head_dim) if read_scale is None else read_scale)
        self.write_scale = float(1.0 if write_scale is None else write_scale)
        self.flags = int(flags)
        self.write_eps = float(write_eps)
        self.nthreads = int(nthreads)
        self.threads_used = 0
        self.len = int(init_len)
        self.n_written = 0
        self.MK = np.zeros((self.U, capacity, head_dim), dtype=np.float64)
        self.MV = np.zeros((self.U, capacity, head_dim), dtype=np.float64)
        if init_len > 0:
            if mk_init is None:
                raise ValueError("mk_init required when init_len > 0")
            self.MK[:, :init_len] = _f64(mk_init).reshape(self.U, init_len, head_dim)
            if mv_init is not None:
                self.MV[:, :init_len] = _f64(mv_init).reshape(self.U, init_len, head_dim)

    # -- state in the caller's layout ------------------------------------------------
    def keys(self) -> np.ndarray:
        return self.MK.reshape(self.B, self.Hkv, self.C, self.d)

    def values(self) -> np.ndarray:
        return self.MV.reshape(self.B, self.Hkv, self.C, self.d)

    # -- steps -------------------------------------------------------------------
    def prefill_stream(self, q, k, v, want_out: bool = True, eta=None):
        """q ``[B, T, Hq, d]``, k, v ``[B, T, Hkv, d]`` -> out ``[B, T, Hq, d]`` (float64).

        ``eta`` ``[B, T, Hkv]``: step size of each token's write (None = all ones)."""
        q = _f64(q)
        k = _f64(k)
        v = _f64(v)
        B, T = q.shape[0], q.shape[1]
        assert q.shape == (self.B, T, self.Hq, self.d), q.shape
        assert k.shape == (self.B, T, self.Hkv, self.d), k.shape
        assert v.shape == (self.B, T, self.Hkv, self.d), v.shape
        # unit-major: unit u = b * Hkv + h ; query heads of kv-head h are h*G .. h*G+G-1
        qu = np.ascontiguousarray(
            q.reshape(B, T, self.Hkv, self.G, self.d).transpose(0, 2, 1, 3, 4)
        ).reshape(self.U, T, self.G, self.d)
        ku = np.ascontiguousarray(k.transpose(0, 2, 1, 3)).reshape(self.U, T, self.d)
        vu = np.ascontiguousarray(v.transpose(0, 2, 1, 3)).reshape(self.U, T, self.d)
        ou = np.empty((self.U, T, self.G, self.d), dtype=np.float64) if want_out else None
        ln = ctypes.c_int64(self.len)
        nw = ctypes.c_int64(self.n_written)
        eu = None
        if eta is not None:
            eta = _f64(eta)
            assert eta.shape == (self.B, T, self.Hkv), eta.shape
            eu = np.ascontiguousarray(eta.transpose(0, 2, 1)).reshape(self.U, T)
        rc = _load().bct_oracle_stream_eps(
            self.U, T, self.G, self.d, self.C, ctypes.byref(ln), ctypes.byref(nw),
            _dptr(self.MK), _dptr(self.MV), _dptr(qu), _dptr(ku), _dptr(vu),
            _dptr(eu) if eu is not None else None,
            _dptr(ou) if want_out else None, self.read_scale, self.write_scale, self.write_eps,
            self.flags, self.nthreads)
        if rc < 0:
            raise RuntimeError("bct_oracle_stream failed")
        self.threads_used = rc
        self.len, self.n_written = ln.value, nw.value
        if not want_out:
            return None
        return np.ascontiguousarray(
            ou.reshape(B, self.Hkv, T, self.G, self.d).transpose(0, 2, 1, 3, 4)
        ).reshape(B, T, self.Hq, self.d)

    def update_kv(self, k, v, eta=None):
        """Algorithm 1 itself (procedure UpdateKV): the write queries k and write key-value vectors v
        ``[B, T, Hkv, d]`` of T tokens go into the state, nothing is read."""
        k = _f64(k)
        q = np.zeros((k.shape[0], k.shape[1], self.Hq, self.d), dtype=np.float64)  # unused: no output is asked for
        self.prefill_stream(q, k, v, want_out=False, eta=eta)

    def decode_step(self, q, k, v, eta=None):
        """q ``[B, Hq, d]``, k, v ``[B, Hkv, d]``, eta ``[B, Hkv]`` or None -> out ``[B, Hq, d]``."""
        q = _f64(q)[:, None]
        k = _f64(k)[:, None]
        v = _f64(v)[:, None]
        return self.prefill_stream(q, k, v, eta=None if eta is None else _f64(eta)[:, None])[:, 0]
