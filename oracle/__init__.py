"""ctypes front end of the CPU oracle (oracle/rmm_oracle.c).

TEST INFRASTRUCTURE.  Only tests/, the smoke check and the benchmark's cpu_baseline /
reference arm may import this package.  It never touches the CUDA library and the CUDA
library never touches it.

Arrays are numpy: dtype uint16 carries raw bf16 bit patterns, float32 and float64 are
themselves.  torch tensors are accepted and viewed without value change (bf16 -> uint16 bits).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rmm_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

BF16, F32, F64 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Building the checker is not using it."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    L = ctypes.CDLL(_LIB)
    i64, dbl, vp, i32 = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
    L.orc_keep_count.restype = i64
    L.orc_keep_count.argtypes = [dbl, i64]
    L.orc_num_threads.restype = i32
    L.orc_set_threads.argtypes = [i32]
    L.orc_score.restype = None
    L.orc_score.argtypes = [vp, i32, i64, i64, i64, i64, vp, vp]
    L.orc_select.restype = dbl
    L.orc_select.argtypes = [vp, i64, i64, vp]
    L.orc_reduced_gemm_rows.restype = None
    L.orc_reduced_gemm_rows.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, i64, i64, i64,
                                        vp, i64, vp, i64, i64]
    L.orc_dense_gemm.restype = None
    L.orc_dense_gemm.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, i64, i64, i64, vp]
    L.orc_round_bf16.restype = dbl
    L.orc_round_bf16.argtypes = [dbl]
    L.orc_attn.restype = None
    L.orc_attn.argtypes = [vp, vp, vp, i32, i64, i64, i64, i64, i64, i64, vp, vp, vp,
                           i32, dbl, dbl, i32, vp, vp, vp, vp]
    L.orc_attn_sets.restype = i32
    L.orc_attn_sets.argtypes = [vp, vp, vp, i32, i64, i64, i64, i64, i64, i64, vp, vp, vp,
                                i32, dbl, dbl, i32, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp]
    _lib = L
    return L


def as_np(x) -> np.ndarray:
    """numpy view of a numpy array or CPU torch tensor; bf16 becomes uint16 bit patterns."""
    if isinstance(x, np.ndarray):
        return x
    import torch  # only to recognise tensors handed in by the tests

    if isinstance(x, torch.Tensor):
        x = x.detach().cpu()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16)
        return x.numpy()
    return np.asarray(x)


def _dt(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float64:
        return F64
    raise TypeError(f"oracle: unsupported dtype {a.dtype}")


def _estr(a: np.ndarray) -> Tuple[int, ...]:
    return tuple(s // a.itemsize for s in a.strides)


def num_threads() -> int:
    return int(_load().orc_num_threads())


def set_threads(n: int) -> None:
    _load().orc_set_threads(int(n))


def keep_count(rho: float, K: int) -> int:
    """|I| = ceil(rho K) (Sec. 3.2); -1 when rho is outside (0, 1] or K < 1."""
    return int(_load().orc_keep_count(float(rho), int(K)))


def score(A) -> Tuple[np.ndarray, np.ndarray]:
    """(energy, score) of the columns of a 2-D matrix: sum of squares and its square root."""
    A = as_np(A)
    assert A.ndim == 2
    M, K = A.shape
    sr, sc = _estr(A)
    e = np.empty(K, np.float64)
    s = np.empty(K, np.float64)
    _load().orc_score(A.ctypes.data, _dt(A), M, K, sr, sc, e.ctypes.data, s.ctypes.data)
    return e, s


def select(key, k: int) -> Tuple[np.ndarray, float]:
    """(ascending index set of the k largest keys with ties to the lower index, kept key mass)."""
    key = np.ascontiguousarray(as_np(key), dtype=np.float64)
    K = key.shape[0]
    assert 1 <= k <= K
    idx = np.empty(k, np.int32)
    kept = _load().orc_select(key.ctypes.data, K, int(k), idx.ctypes.data)
    return idx, float(kept)


def reduced_gemm(A, B, idx, rows: Optional[Tuple[int, int]] = None) -> np.ndarray:
    """Y = A[:, idx] @ B[idx, :] in fp64.  rows=(r0, r1) computes only those rows (others 0)."""
    A, B = as_np(A), as_np(B)
    idx = np.ascontiguousarray(as_np(idx), dtype=np.int32)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    assert idx.size == 0 or (idx.min() >= 0 and idx.max() < K)
    Y = np.zeros((M, N), np.float64)
    r0, r1 = rows if rows is not None else (0, M)
    sra, sca = _estr(A)
    srb, scb = _estr(B)
    _load().orc_reduced_gemm_rows(A.ctypes.data, _dt(A), M, K, sra, sca, B.ctypes.data, _dt(B),
                                  N, srb, scb, idx.ctypes.data, idx.size, Y.ctypes.data, r0, r1)
    return Y


def dense_gemm(A, B) -> np.ndarray:
    """Y = A @ B in fp64 with no index indirection."""
    A, B = as_np(A), as_np(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    Y = np.zeros((M, N), np.float64)
    sra, sca = _estr(A)
    srb, scb = _estr(B)
    _load().orc_dense_gemm(A.ctypes.data, _dt(A), M, K, sra, sca, B.ctypes.data, _dt(B), N, srb, scb,
                           Y.ctypes.data)
    return Y


def round_bf16(x: float) -> float:
    return float(_load().orc_round_bf16(float(x)))


def rmm(A, B, rho: float):
    """The whole operation of Sec. 3.2 on one product: returns (Y, idx, energy)."""
    A = as_np(A)
    e, _ = score(A)
    k = keep_count(rho, A.shape[1])
    idx, _ = select(e, k)
    return reduced_gemm(A, B, idx), idx, e


def attn(Q, K, V, causal: bool, rho_d: float, rho_t: float, round_p: bool = True, want_p: bool = False,
         idx_feat=None, idx_tok=None, rows=None, mask=None):
    """Reduced attention of Sec. 3.3.  Q [B,Hq,Lq,Dh]; K, V [B,Hkv,Lk,Dh] (same dtype).

    idx_feat [B,Hq,kd] / idx_tok [B,Hq,kt] (int32), if given, replace the TopK choice of the feature / token set
    (the formulas for S~ and O~ hold for any set); rows (a list of query rows), if given, restricts the evaluation
    to those rows (with rho_t < 1 the token set must then be given, because token scores need every row).

    mask, if given, is the additive M of P = softmax(S~ + M): an array broadcastable to [B,Hq,Lq,Lk] (-inf hides a key).

    Returns (O [B,Hq,Lq or len(rows),Dh] fp64, idx_feat [B,Hq,kd], idx_tok [B,Hq,kt] or None, P or None):
    the sets are the ones that were used.
    """
    Q, K, V = as_np(Q), as_np(K), as_np(V)
    assert Q.ndim == 4 and K.ndim == 4 and V.ndim == 4 and Q.dtype == K.dtype == V.dtype
    B, Hq, Lq, Dh = Q.shape
    _, Hkv, Lk, _ = K.shape
    assert Hq % Hkv == 0
    kd = keep_count(rho_d, Dh)
    kt = keep_count(rho_t, Lk)
    assert kd >= 1 and kt >= 1
    feat_in = tok_in = rows_in = None
    if idx_feat is not None:
        feat_in = np.ascontiguousarray(as_np(idx_feat), dtype=np.int32)
        assert feat_in.shape == (B, Hq, kd) and feat_in.min() >= 0 and feat_in.max() < Dh
    if idx_tok is not None and rho_t < 1.0:
        tok_in = np.ascontiguousarray(as_np(idx_tok), dtype=np.int32)
        assert tok_in.shape == (B, Hq, kt) and tok_in.min() >= 0 and tok_in.max() < Lk
    nq = Lq
    if rows is not None:
        rows_in = np.ascontiguousarray(np.asarray(rows), dtype=np.int64)
        assert rows_in.ndim == 1 and rows_in.size >= 1 and rows_in.min() >= 0 and rows_in.max() < Lq
        assert rho_t >= 1.0 or tok_in is not None, "token scores need every query row"
        nq = rows_in.size
    O = np.zeros((B, Hq, nq, Dh), np.float64)
    out_feat = np.zeros((B, Hq, kd), np.int32)
    out_tok = np.zeros((B, Hq, kt), np.int32) if rho_t < 1.0 else None
    P = np.zeros((B, Hq, nq, Lk), np.float64) if want_p else None
    s3 = [(ctypes.c_int64 * 4)(*_estr(x)) for x in (Q, K, V)]
    ptr = lambda a: a.ctypes.data if a is not None else None
    mask_in = sm = None
    if mask is not None:
        m = np.asarray(as_np(mask), dtype=np.float64)
        while m.ndim < 4:
            m = m[None]
        assert m.shape[3] == Lk and all(m.shape[a] in (1, n) for a, n in enumerate((B, Hq, Lq)))
        mask_in = np.ascontiguousarray(m)
        full = (mask_in.shape[1] * mask_in.shape[2] * Lk, mask_in.shape[2] * Lk, Lk)
        sm = (ctypes.c_int64 * 3)(*[0 if mask_in.shape[a] == 1 else full[a] for a in range(3)])
    rc = _load().orc_attn_sets(Q.ctypes.data, K.ctypes.data, V.ctypes.data, _dt(Q), B, Hq, Hkv, Lq, Lk, Dh,
                               s3[0], s3[1], s3[2], int(bool(causal)), float(rho_d), float(rho_t),
                               int(bool(round_p)), ptr(feat_in), ptr(tok_in), ptr(rows_in), nq, ptr(mask_in), sm,
                               O.ctypes.data, out_feat.ctypes.data, ptr(out_tok), ptr(P))
    assert rc == 0
    return O, out_feat, out_tok, P


# ------------------------------------------------------------------------------------------------
# 8-bit operands (the paper's appendix "Compatibility with quantization": RMM composed with low-bit inference; the
# e4m3 form).  Plain numpy, written from the format's definition; pinned in tests/test_oracle_pins.py against the
# library's own conversion, hand-made ties, and the exact product of small integer codes.
# ------------------------------------------------------------------------------------------------
E4M3_MAX = 448.0


def e4m3_grid() -> np.ndarray:
    """Every finite non-negative value of the format, ascending: 1 sign, 4 exponent bits (bias 7), 3 mantissa bits, no
    infinities; exponent field 0 holds the subnormals m * 2^-9; the all-ones code is NaN, so the largest value is 448."""
    vals = []
    for e in range(16):
        for m in range(8):
            if e == 15 and m == 7:
                continue                                   # NaN
            vals.append(m * 2.0 ** -9 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7))
    return np.array(vals, dtype=np.float64)


def round_e4m3(x) -> np.ndarray:
    """Nearest value of the format to every element of x (given as float32 numbers), ties to the value with the even
    mantissa code, magnitudes beyond the largest value saturate to +-448.  Returned as float64."""
    x = np.asarray(x, dtype=np.float32).astype(np.float64)
    grid = e4m3_grid()
    a = np.minimum(np.abs(x), E4M3_MAX)
    hi = np.searchsorted(grid, a, side="left")             # first grid value >= a
    hi = np.clip(hi, 0, len(grid) - 1)
    lo = np.clip(hi - 1, 0, len(grid) - 1)
    d_lo, d_hi = a - grid[lo], grid[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))     # codes ascend with the values: even index = even mantissa bit
    out = np.where(pick_hi, grid[hi], grid[lo])
    return np.copysign(out, x)


def quantize_rows_e4m3(A_kept):
    """Per-row dynamic quantisation of already gathered activations A[:, I] (given exactly, as float32-representable
    numbers): step s_i = fp32(max_j |a_ij|) / fp32(448) (1 for an all-zero row), codes q_ij = e4m3(fp32(a_ij / s_i)).
    The division and the step are taken in fp32, which is the precision the decision is defined in.
    Returns (values of the codes as float64 [M, k], steps float32 [M])."""
    A32 = np.asarray(A_kept, dtype=np.float32)
    amax = np.abs(A32).max(axis=1)
    step = np.where(amax > 0, (amax / np.float32(448.0)).astype(np.float32), np.float32(1.0)).astype(np.float32)
    q = round_e4m3((A32 / step[:, None]).astype(np.float32))
    return q, step


def reduced_gemm_q8(A, Bq_values_nk, b_scale: float, idx, rows: Optional[Tuple[int, int]] = None):
    """Y = diag(s) Aq Bq[I, :] * b_scale in fp64, with Aq, s = quantize_rows_e4m3(A[:, I]) and Bq_values_nk the VALUES of
    the weight's codes, stored [N, K].  Returns (Y [M, N] fp64, s)."""
    A = as_np(A)
    if A.dtype == np.uint16:
        A = (A.astype(np.uint32) << 16).view(np.float32)
    idx = np.asarray(as_np(idx), dtype=np.int64)
    q, step = quantize_rows_e4m3(A[:, idx])
    Adeq = q * step.astype(np.float64)[:, None]
    Bdeq = np.ascontiguousarray(np.asarray(Bq_values_nk, dtype=np.float64)[:, idx].T) * float(np.float32(b_scale))
    Y = reduced_gemm(Adeq, Bdeq, np.arange(len(idx), dtype=np.int32), rows=rows)
    return Y, step
