"""Thin ctypes binding of ``libbct_b200.so`` with the names of ``include/bct.h``.

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory (the workspace and the step tensors) and the stream.
There is no CPU fallback: ``load()`` raises when the library has not been built.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

BCT_OK, BCT_ERR_INVALID_ARG, BCT_ERR_UNSUPPORTED, BCT_ERR_STATE, BCT_ERR_CUDA, BCT_ERR_TIMEOUT = range(6)
BCT_F32, BCT_BF16, BCT_BF16_PAIR = 0, 1, 2
FLAG_SKIP_FIRST_WRITE, FLAG_WRITE_THEN_READ, FLAG_DENSE_WRITE, FLAG_OUT_F32, FLAG_PRECISE_READ, FLAG_CUDA_CORES = 1, 2, 4, 8, 16, 32

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libbct_b200.so")

EXPORTS = (
    "bct_version", "bct_last_error", "bct_cache_bytes", "bct_cache_create", "bct_decode_step",
    "bct_prefill_stream", "bct_decode_step_host", "bct_prefill_stream_host", "bct_cache_len",
    "bct_cache_export", "bct_cache_import", "bct_cache_status", "bct_cache_launches", "bct_cache_destroy",
    "bct_cache_tensor_path", "bct_prefill_stream_host_static", "bct_decode_step_eta", "bct_prefill_stream_eta",
    "bct_project_qkv", "bct_layer_scratch_bytes", "bct_layer_forward", "bct_update_kv",
    "bct_cache_status_clear", "bct_cache_rows_rewritten", "bct_selftest_timeout",
    "bct_update_kv_backward", "bct_stack_scratch_bytes", "bct_stack_forward",
)
STATIC_STAGE_BYTES = 8 << 20


class BctParams(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("capacity", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("read_scale", ctypes.c_float), ("write_scale", ctypes.c_float), ("init_len", ctypes.c_int32),
        ("flags", ctypes.c_uint32), ("write_eps", ctypes.c_float), ("max_stream", ctypes.c_int32),
    ]


class BctError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("bct status %d: %s" % (status, message))
        self.status = status


_lib = None


def load() -> ctypes.CDLL:
    """Open the C-ABI library; raise if it is missing (build it with ``python -m paper_2411_15785_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("%s not found: run `python -m paper_2411_15785_b200.build` (no CPU fallback exists)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    pp = ctypes.POINTER(BctParams)
    lib.bct_version.restype = i32
    lib.bct_version.argtypes = []
    lib.bct_last_error.restype = ctypes.c_char_p
    lib.bct_last_error.argtypes = []
    lib.bct_cache_bytes.argtypes = [pp, ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
    lib.bct_cache_create.argtypes = [pp, vp, ctypes.c_size_t, vp, vp, vp, ctypes.POINTER(vp)]
    lib.bct_decode_step.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.bct_prefill_stream.argtypes = [vp, vp, vp, vp, vp, i64, vp]
    lib.bct_decode_step_eta.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.bct_prefill_stream_eta.argtypes = [vp, vp, vp, vp, vp, vp, i64, vp]
    lib.bct_update_kv.argtypes = [vp, vp, vp, vp, i64, vp]
    lib.bct_project_qkv.argtypes = [i64, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.bct_layer_scratch_bytes.argtypes = [vp, i64, ctypes.POINTER(ctypes.c_size_t)]
    lib.bct_layer_forward.argtypes = [vp, vp, vp, vp, vp, i32, vp, vp, ctypes.c_size_t, vp, i64, vp]
    lib.bct_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.bct_prefill_stream_host.argtypes = [vp, vp, vp, vp, vp, i64, vp]
    lib.bct_cache_len.argtypes = [vp, ctypes.POINTER(i32)]
    lib.bct_cache_export.argtypes = [vp, vp, vp, i32, vp]
    lib.bct_cache_import.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.bct_cache_status.argtypes = [vp, vp]
    lib.bct_cache_launches.argtypes = [vp, ctypes.POINTER(i64)]
    lib.bct_cache_destroy.argtypes = [vp]
    lib.bct_cache_tensor_path.argtypes = [vp, ctypes.POINTER(i32)]
    lib.bct_prefill_stream_host_static.argtypes = [vp, vp, vp, vp, vp, i64, vp]
    lib.bct_cache_status_clear.argtypes = [vp, vp]
    lib.bct_cache_rows_rewritten.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint64)]
    lib.bct_selftest_timeout.argtypes = [vp, vp]
    lib.bct_update_kv_backward.argtypes = [vp, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp]
    lib.bct_stack_scratch_bytes.argtypes = [ctypes.POINTER(vp), i32, i64, ctypes.POINTER(ctypes.c_size_t)]
    lib.bct_stack_forward.argtypes = [ctypes.POINTER(vp), i32, vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp),
                                      ctypes.POINTER(vp), vp, ctypes.c_size_t, vp, i64, vp]
    for name in EXPORTS[2:]:
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def last_error() -> str:
    return load().bct_last_error().decode()


def _check(status: int) -> None:
    if status != BCT_OK:
        raise BctError(status, last_error())


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.int32:  # checkpoint words: value-plane bits << 16 | residual-plane bits
        return BCT_BF16_PAIR
    if dt == torch.float32:
        return BCT_F32
    if dt == torch.bfloat16:
        return BCT_BF16
    raise ValueError("dtype must be torch.float32 or torch.bfloat16")


def make_params(batch, n_q_heads, n_kv_heads, head_dim, capacity, dtype, *, read_scale=0.0, write_scale=0.0,
                init_len=0, flags=0, write_eps=0.0, max_stream=1) -> BctParams:
    return BctParams(batch, n_q_heads, n_kv_heads, head_dim, capacity, _dtype_code(dtype), read_scale,
                     write_scale, init_len, flags, write_eps, max_stream)


def cache_bytes(params: BctParams) -> Tuple[int, int]:
    b, a = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(load().bct_cache_bytes(ctypes.byref(params), ctypes.byref(b), ctypes.byref(a)))
    return b.value, a.value


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _check_eta(eta: torch.Tensor, shape) -> None:
    if eta.dtype != torch.float32 or tuple(eta.shape) != tuple(shape) or not eta.is_contiguous() or not eta.is_cuda:
        raise ValueError("eta must be a contiguous float32 device tensor of shape %s" % (tuple(shape),))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def project_qkv(x, w_q, w_wq, w_wv, stream=None, out=None):
    """q = x W_q^T, k = x W_wq^T, v = x W_wv^T: x ``[..., d_model]`` bfloat16 on the device, weights
    ``[features, d_model]``; returns q ``[..., n_q]``, k, v ``[..., n_kv]`` (bfloat16)."""
    lib = load()
    d_model = x.shape[-1]
    n_tokens = x.numel() // d_model
    for t in (x, w_q, w_wq, w_wv):
        if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
            raise ValueError("x and the weights must be contiguous bfloat16 device tensors")
    n_q, n_kv = w_q.shape[0], w_wq.shape[0]
    if out is not None:   # (q, k, v) tensors to write into
        q, k, v = out
    else:
        q = torch.empty(x.shape[:-1] + (n_q,), dtype=torch.bfloat16, device=x.device)
        k = torch.empty(x.shape[:-1] + (n_kv,), dtype=torch.bfloat16, device=x.device)
        v = torch.empty_like(k)
    _check(lib.bct_project_qkv(n_tokens, d_model, n_q, n_kv, x.data_ptr(), w_q.data_ptr(), w_wq.data_ptr(),
                               w_wv.data_ptr(), q.data_ptr(), k.data_ptr(), v.data_ptr(), _stream_ptr(stream)))
    return q, k, v


def stack_forward(caches, x, w_q, w_wq, w_wv, out=None, scratch=None, stream=None):
    """A stack of layers: layer 0 reads x ``[B, T, d_model]``, layer l > 0 the outputs of layer l - 1 as its
    tokens.  caches: list of Cache; w_q, w_wq, w_wv: lists of that layer's weights.  Returns the last layer's
    outputs ``[B, T, Hq, d]``."""
    lib = load()
    n = len(caches)
    T = x.shape[1]
    arr = lambda ptrs: (ctypes.c_void_p * n)(*ptrs)
    hs = arr([c._h.value for c in caches])
    need = ctypes.c_size_t(0)
    _check(lib.bct_stack_scratch_bytes(hs, n, T, ctypes.byref(need)))
    if scratch is None:
        scratch = torch.empty(max(need.value, 256), dtype=torch.uint8, device=x.device)
    last = caches[-1]
    if out is None:
        out = torch.empty((last.B, T, last.Hq, last.d), dtype=torch.bfloat16, device=x.device)
    _check(lib.bct_stack_forward(hs, n, x.data_ptr(), x.shape[2], arr([w.data_ptr() for w in w_q]),
                                 arr([w.data_ptr() for w in w_wq]), arr([w.data_ptr() for w in w_wv]), scratch.data_ptr(),
                                 scratch.numel(), out.data_ptr(), T, _stream_ptr(stream)))
    return out


class Cache:
    """A bounded cache over a torch-allocated workspace.  Methods map 1:1 to the C calls."""

    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, capacity, dtype=torch.bfloat16, *,
                 read_scale=0.0, write_scale=0.0, init_len=0, flags=0, write_eps=0.0, max_stream=1,
                 mk_init: Optional[torch.Tensor] = None, mv_init: Optional[torch.Tensor] = None,
                 device="cuda", stream=None, guard_bytes: int = 0):
        self.lib = load()
        self.params = make_params(batch, n_q_heads, n_kv_heads, head_dim, capacity, dtype,
                                  read_scale=read_scale, write_scale=write_scale, init_len=init_len,
                                  flags=flags, write_eps=write_eps, max_stream=max_stream)
        self.dtype = dtype
        self.out_dtype = torch.float32 if (flags & FLAG_OUT_F32) else dtype
        self.device = torch.device(device)
        self.B, self.Hq, self.Hkv, self.d, self.C = batch, n_q_heads, n_kv_heads, head_dim, capacity
        nbytes, align = cache_bytes(self.params)
        # guard_bytes > 0 (tests): a band of 0xA5 bytes on either side of the workspace, checked by check_guards()
        self._guard = (int(guard_bytes) + align - 1) // align * align
        self.workspace = torch.empty(nbytes + align + 2 * self._guard, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + align - 1) // align * align + self._guard
        self.workspace_bytes = nbytes
        if self._guard:
            self.workspace.fill_(0xA5)
        for t, name in ((mk_init, "mk_init"), (mv_init, "mv_init")):
            if t is not None:
                assert t.is_cuda and t.is_contiguous() and t.dtype == dtype, name
                assert tuple(t.shape) == (batch, n_kv_heads, init_len, head_dim), (name, t.shape)
        self._h = ctypes.c_void_p(None)
        with torch.cuda.device(self.device):
            _check(self.lib.bct_cache_create(ctypes.byref(self.params), self._ws_ptr, nbytes, _ptr(mk_init),
                                             _ptr(mv_init), _stream_ptr(stream), ctypes.byref(self._h)))

    # ---- steps ----------------------------------------------------------------------
    def decode_step(self, q, k, v, out=None, stream=None, eta=None):
        """eta: float32 device tensor [B, Hkv], the step size of each unit's write (None = ones)."""
        if out is None:
            out = torch.empty_like(q, dtype=self.out_dtype)
        if eta is None:
            _check(self.lib.bct_decode_step(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                            _stream_ptr(stream)))
        else:
            _check_eta(eta, (self.B, self.Hkv))
            _check(self.lib.bct_decode_step_eta(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), eta.data_ptr(),
                                                out.data_ptr(), _stream_ptr(stream)))
        return out

    def prefill_stream(self, q, k, v, out=None, want_out=True, stream=None, eta=None):
        """eta: float32 device tensor [B, T, Hkv], the step size of each token's write (None = ones)."""
        T = q.shape[1]
        if out is None and want_out:
            out = torch.empty_like(q, dtype=self.out_dtype)
        if eta is None:
            _check(self.lib.bct_prefill_stream(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), _ptr(out), T,
                                               _stream_ptr(stream)))
        else:
            _check_eta(eta, (self.B, T, self.Hkv))
            _check(self.lib.bct_prefill_stream_eta(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), eta.data_ptr(),
                                                   _ptr(out), T, _stream_ptr(stream)))
        return out

    def update_kv(self, wq, wv, eta=None, stream=None):
        """Algorithm 1's UpdateKV: wq, wv ``[B, T, Hkv, d]`` go into the state, nothing is read."""
        T = wq.shape[1]
        if eta is not None:
            _check_eta(eta, (self.B, T, self.Hkv))
        _check(self.lib.bct_update_kv(self._h, wq.data_ptr(), wv.data_ptr(), _ptr(eta), T, _stream_ptr(stream)))

    def update_kv_backward(self, wq, wv, d_mv, eta=None, want_d_mk=True, want_d_eta=True, out=None, stream=None):
        """Backward of update_kv: d_mv = dL/dMV_N ``[B, Hkv, C, d]`` bfloat16 -> (d_wq, d_wv ``[B, T, Hkv, d]``,
        d_mk ``[B, Hkv, C, d]`` or None, d_eta ``[B, T, Hkv]`` or None), float32.  out: that tuple, to write into."""
        T = wq.shape[1]
        if eta is not None:
            _check_eta(eta, (self.B, T, self.Hkv))
        f32 = dict(dtype=torch.float32, device=self.device)
        if out is not None:
            d_wq, d_wv, d_mk, d_eta = out
        else:
            d_wq, d_wv = torch.empty(tuple(wq.shape), **f32), torch.empty(tuple(wv.shape), **f32)
            d_mk = torch.empty((self.B, self.Hkv, self.C, self.d), **f32) if want_d_mk else None
            d_eta = torch.empty((self.B, T, self.Hkv), **f32) if want_d_eta else None
        _check(self.lib.bct_update_kv_backward(self._h, wq.data_ptr(), wv.data_ptr(), _ptr(eta), d_mv.data_ptr(), T,
                                               d_wq.data_ptr(), d_wv.data_ptr(), _ptr(d_mk), _ptr(d_eta),
                                               _stream_ptr(stream)))
        return d_wq, d_wv, d_mk, d_eta

    def layer_scratch_bytes(self, T: int) -> int:
        n = ctypes.c_size_t(0)
        _check(self.lib.bct_layer_scratch_bytes(self._h, T, ctypes.byref(n)))
        return n.value

    def layer_forward(self, x, w_q, w_wq, w_wv, out=None, want_out=True, eta=None, scratch=None, stream=None):
        """x ``[B, T, d_model]`` bfloat16: projections, then the stream call on their results."""
        T, d_model = x.shape[1], x.shape[2]
        if scratch is None:
            scratch = torch.empty(self.layer_scratch_bytes(T), dtype=torch.uint8, device=self.device)
        if out is None and want_out:
            out = torch.empty((self.B, T, self.Hq, self.d), dtype=self.out_dtype, device=self.device)
        if eta is not None:
            _check_eta(eta, (self.B, T, self.Hkv))
        _check(self.lib.bct_layer_forward(self._h, x.data_ptr(), w_q.data_ptr(), w_wq.data_ptr(), w_wv.data_ptr(),
                                          d_model, _ptr(eta), scratch.data_ptr(), scratch.numel(), _ptr(out), T,
                                          _stream_ptr(stream)))
        return out

    def decode_step_host(self, q, k, v, out, stream=None):
        """q, k, v, out: CPU tensors (pinned for asynchronous copies)."""
        _check(self.lib.bct_decode_step_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                             _stream_ptr(stream)))
        return out

    def prefill_stream_host(self, q, k, v, out, stream=None):
        _check(self.lib.bct_prefill_stream_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), _ptr(out),
                                                q.shape[1], _stream_ptr(stream)))
        return out

    def prefill_stream_host_static(self, q, k, v, out, stream=None):
        """Host tensors in and out, staged in the library's built-in device array (no allocation)."""
        _check(self.lib.bct_prefill_stream_host_static(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                                       out.data_ptr(), q.shape[1], _stream_ptr(stream)))
        return out

    # ---- state ----------------------------------------------------------------------
    @property
    def len(self) -> int:
        n = ctypes.c_int32(0)
        _check(self.lib.bct_cache_len(self._h, ctypes.byref(n)))
        return n.value

    @property
    def tensor_path(self) -> bool:
        n = ctypes.c_int32(0)
        _check(self.lib.bct_cache_tensor_path(self._h, ctypes.byref(n)))
        return bool(n.value)

    @property
    def launches(self) -> int:
        n = ctypes.c_int64(0)
        _check(self.lib.bct_cache_launches(self._h, ctypes.byref(n)))
        return n.value

    def export(self, v_dtype=torch.float32, stream=None):
        shape = (self.B, self.Hkv, self.C, self.d)
        k = torch.empty(shape, dtype=self.dtype, device=self.device)
        v = torch.empty(shape, dtype=v_dtype, device=self.device)
        _check(self.lib.bct_cache_export(self._h, k.data_ptr(), v.data_ptr(), _dtype_code(v_dtype), _stream_ptr(stream)))
        return k, v

    def import_state(self, k, v, length, stream=None):
        vd = _dtype_code(v.dtype) if v is not None else _dtype_code(self.dtype)
        _check(self.lib.bct_cache_import(self._h, _ptr(k), _ptr(v), vd, length, _stream_ptr(stream)))

    def check_guards(self) -> None:
        """Raise if anything wrote outside the workspace (needs guard_bytes > 0 at construction)."""
        if not self._guard:
            return
        torch.cuda.synchronize(self.device)
        lo = self._ws_ptr - self.workspace.data_ptr()
        hi = lo + self.workspace_bytes
        for name, band in (("below", self.workspace[lo - self._guard:lo]), ("above", self.workspace[hi:hi + self._guard])):
            if not bool((band == 0xA5).all()):
                raise AssertionError("guard band %s the workspace was overwritten" % name)

    def status(self, stream=None) -> int:
        return self.lib.bct_cache_status(self._h, _stream_ptr(stream))

    def check_status(self, stream=None) -> None:
        _check(self.status(stream))

    def status_clear(self, stream=None) -> None:
        _check(self.lib.bct_cache_status_clear(self._h, _stream_ptr(stream)))

    def rows_rewritten(self, stream=None) -> int:
        """MV rows stored back by this cache's kernels so far (synchronises the stream)."""
        n = ctypes.c_uint64(0)
        _check(self.lib.bct_cache_rows_rewritten(self._h, _stream_ptr(stream), ctypes.byref(n)))
        return n.value

    def selftest_timeout(self, stream=None) -> None:
        """Launch the block whose bounded wait runs out (reports BCT_ERR_TIMEOUT, site 99)."""
        _check(self.lib.bct_selftest_timeout(self._h, _stream_ptr(stream)))

    def destroy(self) -> None:
        if self._h:
            self.lib.bct_cache_destroy(self._h)
            self._h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
