"""Thin ctypes binding of librmm_b200.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/rmm.h).  Tensors are torch CUDA
tensors used as plain device memory; the current torch stream is the launch stream.  Workspaces are
torch allocations made here (zero-filled once, then cached per device and reused), because the C
library itself never allocates.  There is no fallback: if the shared library is missing or a call is
refused, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librmm_b200.so")

RMM_OK, RMM_ERR_INVALID_ARG, RMM_ERR_UNSUPPORTED, RMM_ERR_WORKSPACE, RMM_ERR_CUDA, RMM_ERR_TIMEOUT, RMM_ERR_BOUNDS = range(7)
RMM_BF16, RMM_F32, RMM_F8E4M3 = 0, 1, 2
RMM_WS_HEADER_BYTES = 4096
_STATUS_NAMES = ["RMM_OK", "RMM_ERR_INVALID_ARG", "RMM_ERR_UNSUPPORTED", "RMM_ERR_WORKSPACE", "RMM_ERR_CUDA",
                 "RMM_ERR_TIMEOUT", "RMM_ERR_BOUNDS"]


class RmmError(RuntimeError):
    def __init__(self, code: int, text: str):
        self.code = code
        name = _STATUS_NAMES[code] if 0 <= code < len(_STATUS_NAMES) else str(code)
        super().__init__(f"{name}: {text}")


class rmm_mat_t(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("batch", ctypes.c_int64),
                ("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("stride_batch", ctypes.c_int64),
                ("stride_row", ctypes.c_int64), ("stride_col", ctypes.c_int64)]


class rmm_attn_desc_t(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int64), ("Hq", ctypes.c_int64), ("Hkv", ctypes.c_int64), ("Lq", ctypes.c_int64),
                ("Lk", ctypes.c_int64), ("Dh", ctypes.c_int64), ("causal", ctypes.c_int32),
                ("rho_d", ctypes.c_double), ("rho_t", ctypes.c_double),
                ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
                ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
                ("mask", ctypes.c_void_p), ("mask_stride", ctypes.c_int64 * 3)]


EXPORTS = ["rmm_keep_count", "rmm_score_workspace_bytes", "rmm_score", "rmm_select_workspace_bytes", "rmm_select",
           "rmm_score_select_workspace_bytes", "rmm_score_select", "rmm_score_select_static",
           "rmm_score_select_static_capacity", "rmm_score_select_static_status", "rmm_reduced_gemm_workspace_bytes",
           "rmm_reduced_gemm", "rmm_reduced_gemm_scored_workspace_bytes", "rmm_reduced_gemm_scored",
           "rmm_reduced_gemm_q8_workspace_bytes", "rmm_reduced_gemm_q8", "rmm_reduced_attn_workspace_bytes", "rmm_reduced_attn",
           "rmm_product_workspace_bytes", "rmm_product", "rmm_product_host_workspace_bytes", "rmm_product_host", "rmm_status_read", "rmm_last_error",
           "rmm_launch_count", "rmm_debug_control", "rmm_profile_kernels", "rmm_profile_count", "rmm_profile_name"]

_lib = None


def lib() -> ctypes.CDLL:
    """Load the shared library; raise if it has not been built (no CPU stand-in exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_13426_b200.build` "
                           "(nvcc, sm_100a); this package has no CPU fallback")
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, dbl, i32, sz, flt = ctypes.c_void_p, ctypes.c_int64, ctypes.c_double, ctypes.c_int, ctypes.c_size_t, ctypes.c_float
    mp = ctypes.POINTER(rmm_mat_t)
    L.rmm_keep_count.argtypes = [dbl, i64, ctypes.POINTER(i64)]
    L.rmm_score_workspace_bytes.argtypes = [mp, i32]
    L.rmm_score_workspace_bytes.restype = sz
    L.rmm_score.argtypes = [mp, i32, vp, vp, vp, sz, vp]
    L.rmm_select_workspace_bytes.argtypes = [i64, i64]
    L.rmm_select_workspace_bytes.restype = sz
    L.rmm_select.argtypes = [vp, i64, i64, dbl, i64, vp, vp, vp, sz, vp]
    L.rmm_score_select_workspace_bytes.argtypes = [mp, i32]
    L.rmm_score_select_workspace_bytes.restype = sz
    L.rmm_score_select.argtypes = [mp, i32, dbl, i64, vp, vp, vp, vp, vp, sz, vp]
    L.rmm_score_select_static.argtypes = [mp, i32, dbl, i64, vp, vp, vp, vp, vp]
    L.rmm_score_select_static_capacity.restype = sz
    L.rmm_score_select_static_status.argtypes = [ctypes.POINTER(i32)]
    L.rmm_reduced_gemm_workspace_bytes.argtypes = [mp, mp, i64, mp]
    L.rmm_reduced_gemm_workspace_bytes.restype = sz
    L.rmm_reduced_gemm.argtypes = [mp, mp, vp, i64, flt, mp, vp, sz, vp]
    L.rmm_reduced_gemm_scored_workspace_bytes.argtypes = [mp, mp, i64, mp]
    L.rmm_reduced_gemm_scored_workspace_bytes.restype = sz
    L.rmm_reduced_gemm_scored.argtypes = [mp, mp, vp, i64, flt, mp, vp, vp, sz, vp]
    L.rmm_reduced_gemm_q8_workspace_bytes.argtypes = [mp, mp, i64, mp]
    L.rmm_reduced_gemm_q8_workspace_bytes.restype = sz
    L.rmm_reduced_gemm_q8.argtypes = [mp, mp, flt, vp, i64, flt, mp, vp, vp, sz, vp]
    L.rmm_reduced_attn_workspace_bytes.argtypes = [ctypes.POINTER(rmm_attn_desc_t)]
    L.rmm_reduced_attn_workspace_bytes.restype = sz
    L.rmm_reduced_attn.argtypes = [ctypes.POINTER(rmm_attn_desc_t), vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.rmm_product_workspace_bytes.argtypes = [mp, mp, mp]
    L.rmm_product_workspace_bytes.restype = sz
    L.rmm_product.argtypes = [mp, mp, dbl, i64, flt, mp, vp, vp, vp, sz, vp]
    L.rmm_product_host_workspace_bytes.argtypes = [i64, i64, i64]
    L.rmm_product_host_workspace_bytes.restype = sz
    L.rmm_product_host.argtypes = [vp, vp, i64, i64, i64, dbl, i32, vp, vp, vp, sz, vp]
    L.rmm_status_read.argtypes = [vp, ctypes.POINTER(i32)]
    L.rmm_last_error.restype = ctypes.c_char_p
    L.rmm_launch_count.restype = i64
    L.rmm_debug_control.argtypes = [ctypes.c_char_p, dbl]
    L.rmm_profile_kernels.argtypes = [vp, vp, i32, ctypes.c_char_p, i32]
    L.rmm_profile_name.argtypes = [i32]
    L.rmm_profile_name.restype = ctypes.c_char_p
    _lib = L
    return L


def _check(rc: int) -> None:
    if rc != RMM_OK:
        raise RmmError(rc, lib().rmm_last_error().decode())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return RMM_BF16
    if t.dtype == torch.float32:
        return RMM_F32
    if t.dtype == torch.float8_e4m3fn:
        return RMM_F8E4M3
    raise RmmError(RMM_ERR_UNSUPPORTED, f"dtype {t.dtype} (bf16, fp32, and e4m3 codes for the 8-bit product)")


def as_mat(t: torch.Tensor) -> rmm_mat_t:
    """Describe a 2-D [rows, cols] or 3-D [batch, rows, cols] CUDA tensor (any strides) as an rmm_mat_t."""
    if not t.is_cuda:
        raise RmmError(RMM_ERR_INVALID_ARG, "tensor is not on a CUDA device")
    if t.dim() == 2:
        b, (r, c), sb, (sr, sc) = 1, t.shape, 0, t.stride()
    elif t.dim() == 3:
        b, r, c = t.shape
        sb, sr, sc = t.stride()
    else:
        raise RmmError(RMM_ERR_INVALID_ARG, "expected a 2-D or 3-D tensor")
    return rmm_mat_t(t.data_ptr(), _dtype_code(t), b, r, c, sb, sr, sc)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


_poison = os.environ.get("RMM_POISON_OUTPUTS", "0") not in ("", "0")


def poison_outputs(on: bool) -> None:
    """Testing aid: when on, every output tensor this module allocates is filled with NaN (floating point) or
    INT32_MIN (indices) before the library is called, so that an element no kernel wrote cannot pass for a result."""
    global _poison
    _poison = bool(on)


def _out(shape, dtype: torch.dtype, device) -> torch.Tensor:
    t = torch.empty(shape, dtype=dtype, device=device)
    if _poison:
        t.fill_(float("nan") if dtype.is_floating_point else torch.iinfo(dtype).min)
    return t


_ws_cache = {}


def workspace(nbytes: int, device: torch.device) -> torch.Tensor:
    """A zero-initialised, cached, growing workspace per device (torch owns the memory)."""
    key = (device.type, device.index if device.index is not None else torch.cuda.current_device())
    ws = _ws_cache.get(key)
    nbytes = max(int(nbytes), RMM_WS_HEADER_BYTES)
    if ws is None or ws.numel() < nbytes:
        ws = torch.zeros(nbytes + 256, dtype=torch.uint8, device=device)
        _ws_cache[key] = ws
    return ws


def _ws_ptr(ws: torch.Tensor) -> Tuple[int, int]:
    p = ws.data_ptr()
    a = (p + 255) // 256 * 256
    return a, ws.numel() - (a - p)


def rmm_keep_count(rho: float, K: int) -> int:
    k = ctypes.c_int64(0)
    _check(lib().rmm_keep_count(float(rho), int(K), ctypes.byref(k)))
    return int(k.value)


def rmm_debug_control(key: str, value: float) -> None:
    """Testing aid: "wait_limit_ms" bounds the device-side waits of later launches, "withhold" makes one kernel family's
    block 0 skip its first tile request (see rmm.h)."""
    _check(lib().rmm_debug_control(key.encode(), float(value)))


def rmm_launch_count() -> int:
    return int(lib().rmm_launch_count())


class KernelTimer:
    """Brackets launches of library kernels whose name contains `name_filter` with CUDA events (one matching launch
    in `every`, at most n of them; rmm_profile_kernels).  Use as a context manager; times_ms() then gives (kernel name, duration) pairs."""

    def __init__(self, n: int, name_filter: str = "", every: int = 1):
        self.n = n
        self.every = every
        self.filter = name_filter.encode()
        self.start = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        self.stop = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        for e in self.start + self.stop:      # torch creates the handle at the first record
            e.record()
        torch.cuda.synchronize()
        self._s = (ctypes.c_void_p * n)(*[e.cuda_event for e in self.start])
        self._e = (ctypes.c_void_p * n)(*[e.cuda_event for e in self.stop])
        self.count = 0
        self.names = []

    def __enter__(self):
        _check(lib().rmm_profile_kernels(self._s, self._e, self.n, self.filter, self.every))
        return self

    def __exit__(self, *exc):
        self.count = int(lib().rmm_profile_count())
        self.names = [lib().rmm_profile_name(i).decode() for i in range(self.count)]
        _check(lib().rmm_profile_kernels(None, None, 0, None, 0))
        return False

    def times_ms(self):
        """[(kernel name, milliseconds)] of the recorded launches (synchronises)."""
        torch.cuda.synchronize()
        return [(self.names[i], self.start[i].elapsed_time(self.stop[i])) for i in range(self.count)]


def rmm_status_read(ws: Optional[torch.Tensor] = None, device=None) -> int:
    """Synchronise the current stream, then read and clear the workspace's device status word."""
    torch.cuda.current_stream().synchronize()
    if ws is None:
        ws = workspace(0, torch.device("cuda", torch.cuda.current_device()) if device is None else device)
    st = ctypes.c_int(0)
    p, _ = _ws_ptr(ws)
    _check(lib().rmm_status_read(p, ctypes.byref(st)))
    return int(st.value)


def rmm_score(A: torch.Tensor, axis: int = 1, want_scores: bool = True, want_energy: bool = True,
              ws: Optional[torch.Tensor] = None):
    """(scores, energy) fp32 [batch, n] (2-D input: [n]); either may be None if not requested."""
    m = as_mat(A)
    n = m.cols if axis == 1 else m.rows
    need = lib().rmm_score_workspace_bytes(ctypes.byref(m), axis)
    if need == 0:
        _check(lib().rmm_score(ctypes.byref(m), axis, None, None, None, 0, None) or RMM_ERR_INVALID_ARG)
    ws = workspace(need, A.device) if ws is None else ws
    p, nb = _ws_ptr(ws)
    shape = (m.batch, n) if A.dim() == 3 else (n,)
    scores = _out(shape, torch.float32, A.device) if want_scores else None
    energy = _out(shape, torch.float32, A.device) if want_energy else None
    _check(lib().rmm_score(ctypes.byref(m), axis, scores.data_ptr() if want_scores else None,
                           energy.data_ptr() if want_energy else None, p, nb, _stream()))
    return scores, energy


def rmm_select(keys: torch.Tensor, rho: float = 0.0, k: int = 0, want_retained: bool = False,
               ws: Optional[torch.Tensor] = None):
    """idx int32 [batch, k] ascending (1-D keys: [k]); with want_retained also the kept key fraction."""
    if keys.dtype != torch.float32 or not keys.is_cuda or not keys.is_contiguous():
        raise RmmError(RMM_ERR_INVALID_ARG, "keys must be a contiguous fp32 CUDA tensor")
    batch, K = (1, keys.shape[0]) if keys.dim() == 1 else keys.shape
    kk = int(k) if k > 0 else rmm_keep_count(rho, K)
    ws = workspace(lib().rmm_select_workspace_bytes(batch, K), keys.device) if ws is None else ws
    p, nb = _ws_ptr(ws)
    idx = _out((batch, kk) if keys.dim() == 2 else (kk,), torch.int32, keys.device)
    ret = _out((batch,), torch.float32, keys.device) if want_retained else None
    _check(lib().rmm_select(keys.data_ptr(), batch, K, float(rho), int(k), idx.data_ptr(),
                            ret.data_ptr() if want_retained else None, p, nb, _stream()))
    return (idx, ret) if want_retained else idx


def rmm_score_select(A: torch.Tensor, rho: float = 0.0, k: int = 0, axis: int = 1, want_scores: bool = False,
                     want_energy: bool = False, want_retained: bool = False, idx: Optional[torch.Tensor] = None,
                     ws: Optional[torch.Tensor] = None):
    """Fused score + top-k.  Returns (idx, scores, energy, retained); unrequested outputs are None."""
    m = as_mat(A)
    n = m.cols if axis == 1 else m.rows
    kk = int(k) if k > 0 else rmm_keep_count(rho, n)
    need = lib().rmm_score_select_workspace_bytes(ctypes.byref(m), axis)
    ws = workspace(need, A.device) if ws is None else ws
    p, nb = _ws_ptr(ws)
    three = A.dim() == 3
    if idx is None:
        idx = _out((m.batch, kk) if three else (kk,), torch.int32, A.device)
    shape = (m.batch, n) if three else (n,)
    scores = _out(shape, torch.float32, A.device) if want_scores else None
    energy = _out(shape, torch.float32, A.device) if want_energy else None
    ret = _out((m.batch,), torch.float32, A.device) if want_retained else None
    _check(lib().rmm_score_select(ctypes.byref(m), axis, float(rho), int(k), idx.data_ptr(),
                                  scores.data_ptr() if want_scores else None,
                                  energy.data_ptr() if want_energy else None,
                                  ret.data_ptr() if want_retained else None, p, nb, _stream()))
    return idx, scores, energy, ret


def rmm_score_select_static(A: torch.Tensor, idx: torch.Tensor, rho: float = 0.0, k: int = 0, axis: int = 1,
                            energy: Optional[torch.Tensor] = None, retained: Optional[torch.Tensor] = None) -> None:
    """Fused score + top-k for callers that cannot allocate: no workspace is passed, the scratch is a device array
    built into the library.  Every buffer is the caller's: idx int32 [batch, k] (or [k]), optional energy fp32
    [batch, n] and retained fp32 [batch] are written in place.  This wrapper itself allocates nothing on the device."""
    m = as_mat(A)
    n = m.cols if axis == 1 else m.rows
    kk = int(k) if k > 0 else rmm_keep_count(rho, n)

    def buf(t, dtype, numel, name):
        if t.dtype != dtype or not t.is_cuda or not t.is_contiguous() or t.numel() != numel:
            raise RmmError(RMM_ERR_INVALID_ARG, f"score_select_static: {name} must be a contiguous {dtype} CUDA tensor of {numel} elements")

    buf(idx, torch.int32, m.batch * kk, "idx")
    if energy is not None:
        buf(energy, torch.float32, m.batch * n, "energy")
    if retained is not None:
        buf(retained, torch.float32, m.batch, "retained")
    _check(lib().rmm_score_select_static(ctypes.byref(m), axis, float(rho), int(k), idx.data_ptr(), None,
                                         energy.data_ptr() if energy is not None else None,
                                         retained.data_ptr() if retained is not None else None, _stream()))


def rmm_score_select_static_capacity() -> int:
    return int(lib().rmm_score_select_static_capacity())


def rmm_score_select_static_status() -> int:
    """Synchronise the current stream, then read and clear the status word of the built-in scratch array."""
    torch.cuda.current_stream().synchronize()
    st = ctypes.c_int(0)
    _check(lib().rmm_score_select_static_status(ctypes.byref(st)))
    return int(st.value)


def rmm_reduced_gemm(A: torch.Tensor, B: torch.Tensor, idx: Optional[torch.Tensor], scale: float = 1.0,
                     out: Optional[torch.Tensor] = None, out_dtype: Optional[torch.dtype] = None,
                     ws: Optional[torch.Tensor] = None, want_energy: bool = False):
    """Y = scale * A[:, idx] @ B[idx, :].  A [M,K] or [b,M,K]; B [K,N] or [b,K,N]; idx int32 [k] or [b,k]
    (None: the unreduced product, k = K, nothing gathered).  want_energy: returns (Y, energy) with energy fp32 [N] or
    [b, N] = column sums of squares of Y as stored (rmm_reduced_gemm_scored)."""
    ma, mb = as_mat(A), as_mat(B)
    if idx is None:
        k = ma.cols
    else:
        if idx.dtype != torch.int32 or not idx.is_cuda or not idx.is_contiguous():
            raise RmmError(RMM_ERR_INVALID_ARG, "idx must be a contiguous int32 CUDA tensor")
        k = idx.shape[-1]
        if idx.numel() != ma.batch * k:
            raise RmmError(RMM_ERR_INVALID_ARG, "idx must hold one index list per batch element of A")
    if out is None:
        dt = out_dtype if out_dtype is not None else A.dtype
        shape = (ma.batch, ma.rows, mb.cols) if A.dim() == 3 else (ma.rows, mb.cols)
        out = _out(shape, dt, A.device)
    my = as_mat(out)
    if want_energy:
        need = lib().rmm_reduced_gemm_scored_workspace_bytes(ctypes.byref(ma), ctypes.byref(mb), k, ctypes.byref(my))
        ws = workspace(need, A.device) if ws is None else ws
        p, nb = _ws_ptr(ws)
        energy = _out((ma.batch, mb.cols) if A.dim() == 3 else (mb.cols,), torch.float32, A.device)
        _check(lib().rmm_reduced_gemm_scored(ctypes.byref(ma), ctypes.byref(mb), idx.data_ptr() if idx is not None else None, k,
                                             float(scale), ctypes.byref(my), energy.data_ptr(), p, nb, _stream()))
        return out, energy
    need = lib().rmm_reduced_gemm_workspace_bytes(ctypes.byref(ma), ctypes.byref(mb), k, ctypes.byref(my))
    ws = workspace(need, A.device) if ws is None else ws
    p, nb = _ws_ptr(ws)
    _check(lib().rmm_reduced_gemm(ctypes.byref(ma), ctypes.byref(mb), idx.data_ptr() if idx is not None else None, k, float(scale),
                                  ctypes.byref(my), p, nb, _stream()))
    return out


def rmm_reduced_gemm_q8(A: torch.Tensor, Bq_nk: torch.Tensor, b_scale: float, idx: torch.Tensor, scale: float = 1.0,
                        out: Optional[torch.Tensor] = None, out_dtype: Optional[torch.dtype] = None, want_scales: bool = False,
                        ws: Optional[torch.Tensor] = None):
    """Reduced product with 8-bit operands.  A bf16 [M, K]; Bq_nk float8_e4m3fn [N, K] (the weight as stored, contraction
    axis contiguous) with one scale b_scale; idx int32 [k].  Returns Y [M, N] (bf16 unless out_dtype says fp32), or
    (Y, a_scale) with want_scales: the per-row quantisation steps of the activations."""
    if Bq_nk.dim() != 2 or Bq_nk.dtype != torch.float8_e4m3fn:
        raise RmmError(RMM_ERR_UNSUPPORTED, "Bq_nk must be a 2-D float8_e4m3fn tensor [N, K]")
    if idx.dtype != torch.int32 or not idx.is_cuda or not idx.is_contiguous() or idx.dim() != 1:
        raise RmmError(RMM_ERR_INVALID_ARG, "idx must be a contiguous 1-D int32 CUDA tensor")
    ma, mb = as_mat(A), as_mat(Bq_nk.t())          # B as a [K, N] matrix whose rows (contraction slices) have stride 1
    k = idx.numel()
    if out is None:
        out = _out((ma.rows, mb.cols), out_dtype if out_dtype is not None else torch.bfloat16, A.device)
    my = as_mat(out)
    need = lib().rmm_reduced_gemm_q8_workspace_bytes(ctypes.byref(ma), ctypes.byref(mb), k, ctypes.byref(my))
    if need == 0:
        raise RmmError(RMM_ERR_UNSUPPORTED, lib().rmm_last_error().decode())
    ws = workspace(need, A.device) if ws is None else ws
    p, nb = _ws_ptr(ws)
    a_scale = _out((ma.rows,), torch.float32, A.device) if want_scales else None
    _check(lib().rmm_reduced_gemm_q8(ctypes.byref(ma), ctypes.byref(mb), float(b_scale), idx.data_ptr(), k, float(scale), ctypes.byref(my),
                                     a_scale.data_ptr() if want_scales else None, p, nb, _stream()))
    return (out, a_scale) if want_scales else out


def rmm_reduced_attn(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, causal: bool, rho_d: float, rho_t: float = 1.0,
                     want_idx: bool = False, ws: Optional[torch.Tensor] = None, mask: Optional[torch.Tensor] = None):
    """Reduced attention.  Q [B,Hq,Lq,Dh], K,V [B,Hkv,Lk,Dh] bf16 with contiguous last dim; mask (optional): additive
    fp32 CUDA tensor [.., Lq, Lk] with up to four dims, size-1 batch / head / row dims shared, contiguous last dim.
    Returns O [B,Hq,Lq,Dh] bf16, or (O, idx_feat, idx_tok) with want_idx (idx_tok None when rho_t == 1)."""
    for t in (Q, K, V):
        if t.dim() != 4 or t.dtype != torch.bfloat16 or not t.is_cuda or t.stride(3) != 1:
            raise RmmError(RMM_ERR_UNSUPPORTED, "Q, K, V must be 4-D bf16 CUDA tensors with a contiguous last dim")
    B, Hq, Lq, Dh = Q.shape
    _, Hkv, Lk, _ = K.shape
    O = _out((B, Hq, Lq, Dh), torch.bfloat16, Q.device)
    d = rmm_attn_desc_t(B, Hq, Hkv, Lq, Lk, Dh, int(bool(causal)), float(rho_d), float(rho_t),
                        (ctypes.c_int64 * 3)(*Q.stride()[:3]), (ctypes.c_int64 * 3)(*K.stride()[:3]),
                        (ctypes.c_int64 * 3)(*V.stride()[:3]), (ctypes.c_int64 * 3)(*O.stride()[:3]),
                        None, (ctypes.c_int64 * 3)(0, 0, 0))
    if mask is not None:
        m = mask
        while m.dim() < 4:
            m = m.unsqueeze(0)
        if (m.dim() != 4 or m.dtype != torch.float32 or not m.is_cuda or m.shape[3] != Lk or (Lk > 1 and m.stride(3) != 1)
                or any(m.shape[a] not in (1, n) for a, n in enumerate((B, Hq, Lq)))):
            raise RmmError(RMM_ERR_INVALID_ARG, "mask must be an fp32 CUDA tensor broadcastable to [B,Hq,Lq,Lk], last dim contiguous")
        d.mask = m.data_ptr()
        d.mask_stride = (ctypes.c_int64 * 3)(*[0 if m.shape[a] == 1 else m.stride(a) for a in range(3)])
    need = lib().rmm_reduced_attn_workspace_bytes(ctypes.byref(d))
    if need == 0:
        raise RmmError(RMM_ERR_INVALID_ARG, "reduced_attn: invalid description (check shapes and retention ratios)")
    ws = workspace(need, Q.device) if ws is None else ws
    p, nb = _ws_ptr(ws)
    idx_feat = idx_tok = None
    if want_idx:
        idx_feat = _out((B, Hq, rmm_keep_count(rho_d, Dh)), torch.int32, Q.device)
        if rho_t < 1.0:
            idx_tok = _out((B, Hq, rmm_keep_count(rho_t, Lk)), torch.int32, Q.device)
    _check(lib().rmm_reduced_attn(ctypes.byref(d), Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(),
                                  idx_feat.data_ptr() if idx_feat is not None else None,
                                  idx_tok.data_ptr() if idx_tok is not None else None, p, nb, _stream()))
    return (O, idx_feat, idx_tok) if want_idx else O


def rmm_product_host(A_host: torch.Tensor, B_host: torch.Tensor, rho: float, Y_host: torch.Tensor,
                     idx_host: Optional[torch.Tensor] = None, copy_B: bool = True,
                     ws: Optional[torch.Tensor] = None, device: Optional[torch.device] = None) -> None:
    """Whole operation on (pinned) host bf16 buffers; asynchronous: synchronise the stream before reading Y_host."""
    M, K = A_host.shape
    _, N = B_host.shape
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    need = lib().rmm_product_host_workspace_bytes(M, K, N)
    ws = workspace(need, device) if ws is None else ws
    p, nb = _ws_ptr(ws)
    _check(lib().rmm_product_host(A_host.data_ptr(), B_host.data_ptr(), M, K, N, float(rho), int(bool(copy_B)),
                                  Y_host.data_ptr(), idx_host.data_ptr() if idx_host is not None else None,
                                  p, nb, _stream()))


def rmm_product(A: torch.Tensor, B: torch.Tensor, rho: float = 0.0, k: int = 0, scale: float = 1.0,
                out: Optional[torch.Tensor] = None, idx: Optional[torch.Tensor] = None, want_retained: bool = False,
                ws: Optional[torch.Tensor] = None):
    """RMM_rho(A, B) of Sec. 3.2 on device tensors in one call: (Y, idx) or (Y, idx, retained)."""
    ma, mb = as_mat(A), as_mat(B)
    kk = int(k) if k > 0 else rmm_keep_count(rho, ma.cols)
    three = A.dim() == 3
    if out is None:
        out = _out((ma.batch, ma.rows, mb.cols) if three else (ma.rows, mb.cols), A.dtype, A.device)
    if idx is None:
        idx = _out((ma.batch, kk) if three else (kk,), torch.int32, A.device)
    elif idx.dtype != torch.int32 or not idx.is_cuda or not idx.is_contiguous() or idx.numel() != ma.batch * kk:
        raise RmmError(RMM_ERR_INVALID_ARG, "idx must be a contiguous int32 CUDA tensor of batch * k elements")
    ret = _out((ma.batch,), torch.float32, A.device) if want_retained else None
    my = as_mat(out)
    need = lib().rmm_product_workspace_bytes(ctypes.byref(ma), ctypes.byref(mb), ctypes.byref(my))
    if need == 0:
        raise RmmError(RMM_ERR_UNSUPPORTED, "rmm_product: operands not covered")
    ws = workspace(need, A.device) if ws is None else ws
    p, nb = _ws_ptr(ws)
    _check(lib().rmm_product(ctypes.byref(ma), ctypes.byref(mb), float(rho), int(k), float(scale), ctypes.byref(my),
                             idx.data_ptr(), ret.data_ptr() if want_retained else None, p, nb, _stream()))
    return (out, idx, ret) if want_retained else (out, idx)


def rmm(A: torch.Tensor, B: torch.Tensor, rho: float, out: Optional[torch.Tensor] = None):
    """RMM_rho(A, B) of Sec. 3.2 on device tensors (rmm_product).  Returns (Y, idx)."""
    return rmm_product(A, B, rho=rho, out=out)
