"""Thin ctypes binding over the C ABI of libspectre.so.

Argument marshalling only: every step of the path runs in the CUDA kernels.
Function names are those of include/spectre.h.  PyTorch appears here for device
memory (tensors, workspace) and the current stream, nothing else.  If the
shared library is missing the import of any entry point raises: there is no CPU
or PyTorch fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libspectre.so")
_lib = None

SPECTRE_OK = 0
SPECTRE_ERR_INVALID_ARG = 1
SPECTRE_ERR_UNSUPPORTED = 2
SPECTRE_ERR_WORKSPACE = 3
SPECTRE_ERR_CUDA = 4
SPECTRE_ERR_TIMEOUT = 5
SPECTRE_ERR_RANGE = 6
SPECTRE_F32 = 0
SPECTRE_BF16 = 1
SPECTRE_F16 = 2

EXPORTS = [
    "spectre_create", "spectre_destroy", "spectre_status_string", "spectre_last_error", "spectre_poll_status",
    "spectre_selftest_wait_timeout",
    "spectre_gate_workspace_bytes", "spectre_gate", "spectre_gate_static_max_bytes", "spectre_gate_static",
    "spectre_mixer_workspace_bytes", "spectre_mixer_forward",
    "spectre_wavelet_refine",
    "spectre_prefill_workspace_bytes", "spectre_prefix_cache_prefill", "spectre_prefix_cache_append",
    "spectre_decode_workspace_bytes", "spectre_prefix_cache_decode_step",
    "spectre_readout_workspace_bytes", "spectre_prefix_cache_readout",
    "spectre_mixer_backward_workspace_bytes", "spectre_mixer_backward",
    "spectre_project_workspace_bytes", "spectre_project_qv",
]
DECODE_MAX_ROWS = 4


class SpectreError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"spectre status {status}: {msg}")
        self.status = status


class Act(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("B", C.c_int32), ("L", C.c_int32),
                ("H", C.c_int32), ("D", C.c_int32), ("stride_b", C.c_int64), ("stride_l", C.c_int64),
                ("stride_h", C.c_int64)]


class GateParams(C.Structure):
    _fields_ = [("wdtype", C.c_int32), ("hidden", C.c_int32), ("toeplitz_r", C.c_int32),
                ("shared_across_heads", C.c_int32), ("ln_gamma", C.c_void_p), ("ln_beta", C.c_void_p),
                ("ln_eps", C.c_float), ("W1", C.c_void_p), ("b1", C.c_void_p), ("W2", C.c_void_p),
                ("b2", C.c_void_p), ("modrelu_bias", C.c_void_p), ("toeplitz", C.c_void_p)]


class Wavelet(C.Structure):
    _fields_ = [("levels", C.c_int32), ("hidden", C.c_int32), ("wdtype", C.c_int32),
                ("shared_across_heads", C.c_int32), ("level_gates", C.c_void_p), ("qbar", C.c_void_p),
                ("Ww1", C.c_void_p), ("bw1", C.c_void_p), ("Ww2", C.c_void_p), ("bw2", C.c_void_p),
                ("skip", C.c_void_p)]


class Cache(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("D", C.c_int32), ("N_max", C.c_int32),
                ("buf_dtype", C.c_int32), ("reserved", C.c_int32), ("prefix_fft", C.c_void_p),
                ("V_buf", C.c_void_p), ("Q_buf", C.c_void_p), ("sum_q", C.c_void_p)]


def lib():
    """Loads libspectre.so (built in-tree by paper_2502_18394_b200.build); fails loudly if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2502_18394_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(_LIB_PATH)
    L.spectre_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
    L.spectre_destroy.argtypes = [C.c_void_p]
    L.spectre_poll_status.argtypes = [C.c_void_p]
    L.spectre_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_void_p]
    L.spectre_selftest_wait_timeout.restype = C.c_int
    L.spectre_status_string.argtypes = [C.c_int]
    L.spectre_status_string.restype = C.c_char_p
    L.spectre_last_error.restype = C.c_char_p
    L.spectre_gate_workspace_bytes.argtypes = [C.c_void_p] + [C.c_int32] * 5
    L.spectre_gate_workspace_bytes.restype = C.c_size_t
    L.spectre_gate.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Act), C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                               C.c_float, C.POINTER(GateParams), C.c_int32, C.c_void_p, C.c_int64, C.c_void_p,
                               C.c_void_p, C.c_void_p, C.c_size_t]
    L.spectre_gate_static_max_bytes.restype = C.c_size_t
    L.spectre_gate_static.argtypes = L.spectre_gate.argtypes[:-2]
    L.spectre_mixer_workspace_bytes.argtypes = [C.c_void_p] + [C.c_int32] * 6
    L.spectre_mixer_workspace_bytes.restype = C.c_size_t
    L.spectre_mixer_forward.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Act), C.c_void_p, C.POINTER(Act), C.c_int32,
                                        C.POINTER(Wavelet), C.c_void_p, C.c_size_t]
    L.spectre_wavelet_refine.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Act), C.POINTER(Act), C.POINTER(Wavelet)]
    L.spectre_prefill_workspace_bytes.argtypes = [C.c_void_p] + [C.c_int32] * 4
    L.spectre_prefill_workspace_bytes.restype = C.c_size_t
    L.spectre_prefix_cache_prefill.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Cache), C.POINTER(Act), C.POINTER(Act),
                                               C.c_void_p, C.c_size_t]
    L.spectre_prefix_cache_append.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Cache), C.c_void_p, C.c_void_p,
                                              C.c_int64]
    L.spectre_project_workspace_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
    L.spectre_project_workspace_bytes.restype = C.c_size_t
    L.spectre_project_qv.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Act), C.c_void_p, C.c_void_p, C.c_int32,
                                     C.POINTER(Act), C.POINTER(Act), C.c_void_p, C.c_void_p, C.c_size_t]
    L.spectre_mixer_backward_workspace_bytes.argtypes = [C.c_void_p] + [C.c_int32] * 6
    L.spectre_mixer_backward_workspace_bytes.restype = C.c_size_t
    L.spectre_mixer_backward.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Act), C.POINTER(Act), C.c_void_p,
                                         C.POINTER(Act), C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t]
    L.spectre_readout_workspace_bytes.argtypes = [C.c_void_p] + [C.c_int32] * 4
    L.spectre_readout_workspace_bytes.restype = C.c_size_t
    L.spectre_prefix_cache_readout.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Cache), C.c_void_p, C.POINTER(Act),
                                               C.c_void_p, C.c_size_t]
    L.spectre_decode_workspace_bytes.argtypes = [C.c_void_p] + [C.c_int32] * 6
    L.spectre_decode_workspace_bytes.restype = C.c_size_t
    L.spectre_prefix_cache_decode_step.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Cache), C.c_void_p, C.c_void_p,
                                                   C.c_int64, C.POINTER(GateParams), C.POINTER(C.c_int32), C.c_int32,
                                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t]
    _lib = L
    return L


def _check(status: int):
    if status != SPECTRE_OK:
        L = lib()
        raise SpectreError(status, f"{L.spectre_status_string(status).decode()}: {L.spectre_last_error().decode()}")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SPECTRE_F32
    if t.dtype == torch.bfloat16:
        return SPECTRE_BF16
    if t.dtype == torch.float16:
        return SPECTRE_F16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def act(t: torch.Tensor) -> Act:
    """Descriptor of a [B, L, H, D] tensor (any strides with D contiguous)."""
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("activation must be [B, L, H, D] with D contiguous")
    return Act(t.data_ptr(), _dtype_code(t), t.shape[0], t.shape[1], t.shape[2], t.shape[3],
               t.stride(0), t.stride(1), t.stride(2))


class Context:
    """Owns a spectre_ctx*; `device` is the CUDA device index."""

    def __init__(self, device: int = 0):
        self.handle = C.c_void_p()
        _check(lib().spectre_create(C.byref(self.handle), device))
        self.device = device

    def poll_status(self):
        """Raises SpectreError(SPECTRE_ERR_TIMEOUT) if a kernel gave up on a bounded wait, or
        SpectreError(SPECTRE_ERR_RANGE) if a 16-bit tensor-core mixer overflowed (call after a sync)."""
        _check(lib().spectre_poll_status(self.handle))

    def selftest_wait_timeout(self):
        """Enqueues the diagnostic kernel whose bounded wait runs out by construction."""
        _check(lib().spectre_selftest_wait_timeout(self.handle, _stream()))

    def close(self):
        if self.handle:
            lib().spectre_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _gate_struct(p: dict, keep: list) -> GateParams:
    tz = p.get("toeplitz")
    r = 0 if tz is None else (tz.shape[-2] - 1) // 2
    keep.extend([p["ln_gamma"], p["ln_beta"], p["W1"], p["b1"], p["W2"], p["b2"], p.get("modrelu_bias"), tz])
    return GateParams(_dtype_code(p["W1"]), int(p["hidden"]), r, int(p.get("shared_across_heads", 0)),
                      p["ln_gamma"].data_ptr(), p["ln_beta"].data_ptr(), float(p["ln_eps"]),
                      p["W1"].data_ptr(), p["b1"].data_ptr(), p["W2"].data_ptr(), p["b2"].data_ptr(),
                      None if p.get("modrelu_bias") is None else p["modrelu_bias"].data_ptr(),
                      None if tz is None else tz.data_ptr())


def _wavelet_struct(w: dict | None, keep: list):
    if w is None:
        return None
    keep.append(w)
    g = w.get("level_gates")
    wd = SPECTRE_F32 if w.get("Ww1") is None else _dtype_code(w["Ww1"])
    return Wavelet(int(w["levels"]), int(w.get("hidden", 0)), wd, int(w.get("shared_across_heads", 0)),
                   None if g is None else g.data_ptr(),
                   None if w.get("qbar") is None else w["qbar"].data_ptr(),
                   None if w.get("Ww1") is None else w["Ww1"].data_ptr(),
                   None if w.get("bw1") is None else w["bw1"].data_ptr(),
                   None if w.get("Ww2") is None else w["Ww2"].data_ptr(),
                   None if w.get("bw2") is None else w["bw2"].data_ptr(),
                   None if w.get("skip") is None else w["skip"].data_ptr())


def _workspace(nbytes: int, device) -> torch.Tensor | None:
    return torch.empty(max(nbytes, 16), dtype=torch.uint8, device=device) if nbytes > 0 else None


def spectre_gate_workspace_bytes(ctx: Context, B, H, D, n_fft, toeplitz_r=0) -> int:
    return lib().spectre_gate_workspace_bytes(ctx.handle, B, H, D, n_fft, toeplitz_r)


def spectre_gate(ctx: Context, params: dict, n_fft: int, q: torch.Tensor | None = None,
                 sum_q: torch.Tensor | None = None, inv_count: float = 0.0, shift: torch.Tensor | None = None,
                 shift_all: int = 0, g_out: torch.Tensor | None = None, qbar_out: torch.Tensor | None = None,
                 workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """g[B,H,K,2] = gate(...) (Sec. 3.2 step 3).  Allocates g_out / workspace with torch when not given."""
    ref = q if q is not None else sum_q
    if q is not None:
        B, _, H, D = q.shape
    else:
        B, H, D = sum_q.shape
    K = n_fft // 2 + 1
    keep: list = []
    gp = _gate_struct(params, keep)
    if g_out is None:
        g_out = torch.empty((B, H, K, 2), dtype=torch.float32, device=ref.device)
    if workspace is None:
        workspace = _workspace(spectre_gate_workspace_bytes(ctx, B, H, D, n_fft, gp.toeplitz_r), ref.device)
    a = act(q) if q is not None else None
    _check(lib().spectre_gate(ctx.handle, _stream(stream), None if a is None else C.byref(a), _ptr(sum_q), B, H, D,
                              float(inv_count), C.byref(gp), n_fft, _ptr(shift), int(shift_all), _ptr(g_out),
                              _ptr(qbar_out), _ptr(workspace), 0 if workspace is None else workspace.numel()))
    return g_out


def spectre_gate_static_max_bytes() -> int:
    return lib().spectre_gate_static_max_bytes()


def spectre_gate_static(ctx: Context, params: dict, n_fft: int, g_out: torch.Tensor, q: torch.Tensor | None = None,
                        sum_q: torch.Tensor | None = None, inv_count: float = 0.0,
                        shift: torch.Tensor | None = None, shift_all: int = 0,
                        qbar_out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """spectre_gate with the scratch inside the library: for callers that may not allocate device
    memory where the gate runs.  Nothing is allocated here either, so the output tensor g_out
    [B,H,K,2] is a required argument.  Calls on one device share the scratch: do not overlap them."""
    if q is not None:
        B, _, H, D = q.shape
    else:
        B, H, D = sum_q.shape
    keep: list = []
    gp = _gate_struct(params, keep)
    a = act(q) if q is not None else None
    _check(lib().spectre_gate_static(ctx.handle, _stream(stream), None if a is None else C.byref(a), _ptr(sum_q),
                                     B, H, D, float(inv_count), C.byref(gp), n_fft, _ptr(shift), int(shift_all),
                                     _ptr(g_out), _ptr(qbar_out)))
    return g_out


def spectre_mixer_workspace_bytes(ctx: Context, B, L, H, D, n_fft, dtype_code) -> int:
    return lib().spectre_mixer_workspace_bytes(ctx.handle, B, L, H, D, n_fft, dtype_code)


def spectre_mixer_forward(ctx: Context, v: torch.Tensor, g: torch.Tensor, y: torch.Tensor | None = None,
                          n_fft: int | None = None, wrm: dict | None = None,
                          workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Y = irfft(g * rfft(V)) per head (Sec. 3.2 steps 2, 4)."""
    B, L, H, D = v.shape
    n = L if n_fft is None else n_fft
    if y is None:
        y = torch.empty_like(v)
    if workspace is None:
        workspace = _workspace(spectre_mixer_workspace_bytes(ctx, B, L, H, D, n, _dtype_code(v)), v.device)
    keep: list = []
    w = _wavelet_struct(wrm, keep)
    av, ay = act(v), act(y)
    _check(lib().spectre_mixer_forward(ctx.handle, _stream(stream), C.byref(av), _ptr(g), C.byref(ay), n,
                                       None if w is None else C.byref(w), _ptr(workspace),
                                       0 if workspace is None else workspace.numel()))
    return y


def spectre_wavelet_refine(ctx: Context, y_in: torch.Tensor, wrm: dict, y_out: torch.Tensor | None = None,
                           stream=None) -> torch.Tensor:
    """Y_out = Y_in + W^-1(s * W Y_in) (Sec. 3.5)."""
    if y_out is None:
        y_out = torch.empty_like(y_in)
    keep: list = []
    w = _wavelet_struct(wrm, keep)
    ai, ao = act(y_in), act(y_out)
    _check(lib().spectre_wavelet_refine(ctx.handle, _stream(stream), C.byref(ai), C.byref(ao), C.byref(w)))
    return y_out


class PrefixCache:
    """Caller-owned cache tensors of Alg. 1 (allocated with torch) plus their C descriptor."""

    def __init__(self, B, H, D, N_max, dtype=torch.bfloat16, device="cuda"):
        K = N_max // 2 + 1
        self.B, self.H, self.D, self.N_max = B, H, D, N_max
        self.prefix_fft = torch.zeros((B, H, K, D, 2), dtype=torch.float32, device=device)
        self.V_buf = torch.zeros((B, N_max, H, D), dtype=dtype, device=device)
        self.Q_buf = torch.zeros((B, N_max, H, D), dtype=dtype, device=device)
        self.sum_q = torch.zeros((B, H, D), dtype=torch.float32, device=device)

    def struct(self) -> Cache:
        return Cache(self.B, self.H, self.D, self.N_max, _dtype_code(self.V_buf), 0, self.prefix_fft.data_ptr(),
                     self.V_buf.data_ptr(), self.Q_buf.data_ptr(), self.sum_q.data_ptr())


def spectre_prefill_workspace_bytes(ctx: Context, B, H, D, N_max) -> int:
    return lib().spectre_prefill_workspace_bytes(ctx.handle, B, H, D, N_max)


def spectre_prefix_cache_prefill(ctx: Context, cache: PrefixCache, q: torch.Tensor, v: torch.Tensor,
                                 workspace: torch.Tensor | None = None, stream=None) -> None:
    """PreFill of Alg. 1."""
    if workspace is None:
        workspace = _workspace(spectre_prefill_workspace_bytes(ctx, cache.B, cache.H, cache.D, cache.N_max), v.device)
    cs = cache.struct()
    aq, av = act(q), act(v)
    _check(lib().spectre_prefix_cache_prefill(ctx.handle, _stream(stream), C.byref(cs), C.byref(aq), C.byref(av),
                                              _ptr(workspace), 0 if workspace is None else workspace.numel()))


def spectre_prefix_cache_append(ctx: Context, cache: PrefixCache, q_t: torch.Tensor, v_t: torch.Tensor, t: int,
                                stream=None) -> None:
    """DecodeStep of Alg. 1, steps (a)-(b)."""
    if not (q_t.is_contiguous() and v_t.is_contiguous()):
        raise ValueError("q_t and v_t must be contiguous [B, H, D]")
    cs = cache.struct()
    _check(lib().spectre_prefix_cache_append(ctx.handle, _stream(stream), C.byref(cs), _ptr(q_t), _ptr(v_t), int(t)))


def spectre_decode_workspace_bytes(ctx: Context, B, H, D, N_max, nrows, toeplitz_r=0) -> int:
    return lib().spectre_decode_workspace_bytes(ctx.handle, B, H, D, N_max, nrows, toeplitz_r)


def spectre_prefix_cache_decode_step(ctx: Context, cache: PrefixCache, q_t: torch.Tensor, v_t: torch.Tensor, t: int,
                                     params: dict, rows, y_rows: torch.Tensor | None = None,
                                     g_out: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                                     stream=None):
    """Whole DecodeStep of Alg. 1 with the listed read-out rows.  Returns (y_rows [B,len(rows),H,D], g [B,H,K,2])."""
    if not (q_t.is_contiguous() and v_t.is_contiguous()):
        raise ValueError("q_t and v_t must be contiguous [B, H, D]")
    rows = [int(r) for r in rows]
    keep: list = []
    gp = _gate_struct(params, keep)
    K = cache.N_max // 2 + 1
    if y_rows is None:
        y_rows = torch.empty((cache.B, len(rows), cache.H, cache.D), dtype=v_t.dtype, device=v_t.device)
    if g_out is None:
        g_out = torch.empty((cache.B, cache.H, K, 2), dtype=torch.float32, device=v_t.device)
    if workspace is None:
        workspace = _workspace(spectre_decode_workspace_bytes(ctx, cache.B, cache.H, cache.D, cache.N_max,
                                                              max(1, min(len(rows), DECODE_MAX_ROWS)), gp.toeplitz_r),
                               v_t.device)
    cs = cache.struct()
    arr = (C.c_int32 * max(1, len(rows)))(*rows)
    _check(lib().spectre_prefix_cache_decode_step(ctx.handle, _stream(stream), C.byref(cs), _ptr(q_t), _ptr(v_t), int(t),
                                                  C.byref(gp), arr, len(rows), _ptr(y_rows), _ptr(g_out),
                                                  _ptr(workspace), 0 if workspace is None else workspace.numel()))
    return y_rows, g_out


def spectre_project_workspace_bytes(ctx: Context, H, D) -> int:
    return lib().spectre_project_workspace_bytes(ctx.handle, H, D)


def spectre_project_qv(ctx: Context, x: torch.Tensor, Wq: torch.Tensor, Wv: torch.Tensor, q: torch.Tensor | None = None,
                       v: torch.Tensor | None = None, sum_q: torch.Tensor | None = None, need_sum: bool = True,
                       workspace: torch.Tensor | None = None, stream=None):
    """Q = X Wq, V = X Wv per head (Eq. 2) and sum_q = sum over the sequence of Q.  Returns (q, v, sum_q)."""
    B, L, H, D = x.shape
    if Wq.dtype != Wv.dtype or not (Wq.is_contiguous() and Wv.is_contiguous()):
        raise ValueError("Wq and Wv must be contiguous and of one dtype")
    q = torch.empty_like(x) if q is None else q
    v = torch.empty_like(x) if v is None else v
    if sum_q is None and need_sum:
        sum_q = torch.empty((B, H, D), dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = _workspace(spectre_project_workspace_bytes(ctx, H, D), x.device)
    ax, aq, av = act(x), act(q), act(v)
    _check(lib().spectre_project_qv(ctx.handle, _stream(stream), C.byref(ax), _ptr(Wq), _ptr(Wv), _dtype_code(Wq),
                                    C.byref(aq), C.byref(av), _ptr(sum_q), _ptr(workspace),
                                    0 if workspace is None else workspace.numel()))
    return q, v, sum_q


def spectre_mixer_backward_workspace_bytes(ctx: Context, B, L, H, D, n_fft, dtype_code) -> int:
    return lib().spectre_mixer_backward_workspace_bytes(ctx.handle, B, L, H, D, n_fft, dtype_code)


def spectre_mixer_backward(ctx: Context, v: torch.Tensor, dy: torch.Tensor, g: torch.Tensor, n_fft: int | None = None,
                           need_dv: bool = True, need_dg: bool = True, workspace: torch.Tensor | None = None,
                           stream=None):
    """Gradients of <dy, mixer(v, g)>: (dv like v or None, dg [B,H,K,2] float32 or None)."""
    B, L, H, D = v.shape
    n = L if n_fft is None else n_fft
    dv = torch.empty_like(v) if need_dv else None
    dg = torch.empty((B, H, n // 2 + 1, 2), dtype=torch.float32, device=v.device) if need_dg else None
    if workspace is None:
        workspace = _workspace(spectre_mixer_backward_workspace_bytes(ctx, B, L, H, D, n, _dtype_code(v)), v.device)
    av, ady = act(v), act(dy)
    adv = act(dv) if need_dv else None
    _check(lib().spectre_mixer_backward(ctx.handle, _stream(stream), C.byref(av), C.byref(ady), _ptr(g),
                                        None if adv is None else C.byref(adv), _ptr(dg), n, _ptr(workspace),
                                        0 if workspace is None else workspace.numel()))
    return dv, dg


def spectre_readout_workspace_bytes(ctx: Context, B, H, D, N_max) -> int:
    return lib().spectre_readout_workspace_bytes(ctx.handle, B, H, D, N_max)


def spectre_prefix_cache_readout(ctx: Context, cache: PrefixCache, g: torch.Tensor, y: torch.Tensor | None = None,
                                 workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Whole-window read-out irfft(g * prefix_fft) (Sec. 3.3.2 step e) -> [B, N_max, H, D]."""
    if y is None:
        y = torch.empty((cache.B, cache.N_max, cache.H, cache.D), dtype=cache.V_buf.dtype, device=g.device)
    if workspace is None:
        workspace = _workspace(spectre_readout_workspace_bytes(ctx, cache.B, cache.H, cache.D, cache.N_max), g.device)
    cs = cache.struct()
    ay = act(y)
    _check(lib().spectre_prefix_cache_readout(ctx.handle, _stream(stream), C.byref(cs), _ptr(g), C.byref(ay),
                                              _ptr(workspace), 0 if workspace is None else workspace.numel()))
    return y


# ---- pre-marshalled calls ---------------------------------------------------------------
# A launch loop that rebuilds ctypes structures every step spends more host time than the
# kernels take.  These objects marshal once and replay the identical C call.
class PreparedCall:
    def __init__(self, fn, args, keep):
        self._fn, self._args, self._keep = fn, args, keep

    def __call__(self):
        st = self._fn(*self._args)
        if st != SPECTRE_OK:
            _check(st)


def prepare_gate(ctx: Context, params: dict, n_fft: int, q: torch.Tensor, g_out: torch.Tensor,
                 workspace: torch.Tensor, qbar_out: torch.Tensor | None = None, shift_all: int = 0,
                 stream=None) -> PreparedCall:
    B, _, H, D = q.shape
    keep: list = [q, g_out, workspace, qbar_out]
    gp = _gate_struct(params, keep)
    a = act(q)
    keep += [gp, a]
    args = (ctx.handle, _stream(stream), C.byref(a), None, B, H, D, C.c_float(0.0), C.byref(gp), n_fft, None,
            int(shift_all), _ptr(g_out), _ptr(qbar_out), _ptr(workspace), workspace.numel())
    return PreparedCall(lib().spectre_gate, args, keep)


def prepare_mixer_forward(ctx: Context, v: torch.Tensor, g: torch.Tensor, y: torch.Tensor, n_fft: int | None = None,
                          wrm: dict | None = None, workspace: torch.Tensor | None = None, stream=None) -> PreparedCall:
    n = v.shape[1] if n_fft is None else n_fft
    keep: list = [v, g, y, workspace]
    w = _wavelet_struct(wrm, keep)
    av, ay = act(v), act(y)
    keep += [w, av, ay]
    args = (ctx.handle, _stream(stream), C.byref(av), _ptr(g), C.byref(ay), n, None if w is None else C.byref(w),
            _ptr(workspace), 0 if workspace is None else workspace.numel())
    return PreparedCall(lib().spectre_mixer_forward, args, keep)


def prepare_decode_step(ctx: Context, cache: PrefixCache, q_t: torch.Tensor, v_t: torch.Tensor, t: int, params: dict,
                        rows, y_rows: torch.Tensor, g_out: torch.Tensor, workspace: torch.Tensor,
                        stream=None) -> PreparedCall:
    cs = cache.struct()
    keep: list = [cache, q_t, v_t, cs, y_rows, g_out, workspace]
    gp = _gate_struct(params, keep)
    arr = (C.c_int32 * len(rows))(*[int(r) for r in rows])
    keep += [gp, arr]
    args = (ctx.handle, _stream(stream), C.byref(cs), _ptr(q_t), _ptr(v_t), int(t), C.byref(gp), arr, len(rows),
            _ptr(y_rows), _ptr(g_out), _ptr(workspace), workspace.numel())
    return PreparedCall(lib().spectre_prefix_cache_decode_step, args, keep)


def prepare_project_qv(ctx: Context, x: torch.Tensor, Wq: torch.Tensor, Wv: torch.Tensor, q: torch.Tensor,
                       v: torch.Tensor, sum_q: torch.Tensor, workspace: torch.Tensor, stream=None) -> PreparedCall:
    ax, aq, av = act(x), act(q), act(v)
    keep = [x, Wq, Wv, q, v, sum_q, workspace, ax, aq, av]
    args = (ctx.handle, _stream(stream), C.byref(ax), _ptr(Wq), _ptr(Wv), _dtype_code(Wq), C.byref(aq), C.byref(av),
            _ptr(sum_q), _ptr(workspace), workspace.numel())
    return PreparedCall(lib().spectre_project_qv, args, keep)


def prepare_gate_from_sum(ctx: Context, params: dict, n_fft: int, sum_q: torch.Tensor, inv_count: float,
                          g_out: torch.Tensor, workspace: torch.Tensor, qbar_out: torch.Tensor | None = None,
                          shift_all: int = 0, stream=None) -> PreparedCall:
    B, H, D = sum_q.shape
    keep: list = [sum_q, g_out, workspace, qbar_out]
    gp = _gate_struct(params, keep)
    keep += [gp]
    args = (ctx.handle, _stream(stream), None, _ptr(sum_q), B, H, D, C.c_float(inv_count), C.byref(gp), n_fft, None,
            int(shift_all), _ptr(g_out), _ptr(qbar_out), _ptr(workspace), workspace.numel())
    return PreparedCall(lib().spectre_gate, args, keep)


def prepare_mixer_backward(ctx: Context, v: torch.Tensor, dy: torch.Tensor, g: torch.Tensor, dv: torch.Tensor,
                           dg: torch.Tensor, workspace: torch.Tensor, n_fft: int | None = None,
                           stream=None) -> PreparedCall:
    n = v.shape[1] if n_fft is None else n_fft
    av, ady, adv = act(v), act(dy), act(dv)
    keep = [v, dy, g, dv, dg, workspace, av, ady, adv]
    args = (ctx.handle, _stream(stream), C.byref(av), C.byref(ady), _ptr(g), C.byref(adv), _ptr(dg), n,
            _ptr(workspace), workspace.numel())
    return PreparedCall(lib().spectre_mixer_backward, args, keep)


def prepare_append(ctx: Context, cache: PrefixCache, q_t: torch.Tensor, v_t: torch.Tensor, t: int,
                   stream=None) -> PreparedCall:
    cs = cache.struct()
    keep = [cache, q_t, v_t, cs]
    args = (ctx.handle, _stream(stream), C.byref(cs), _ptr(q_t), _ptr(v_t), int(t))
    return PreparedCall(lib().spectre_prefix_cache_append, args, keep)
