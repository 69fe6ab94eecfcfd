"""fp64 CPU oracle for block-sparse spatiotemporal attention -- TEST INFRASTRUCTURE.

Thin ctypes wrapper over ``sva_oracle.c`` (plain C, fp64, OpenMP over rows).  Only the
tests, the smoke check and the bench's ``cpu_baseline`` / ``--impl reference`` legs may
import this package; the CUDA path never does, and this package imports nothing from it.

All tensors are numpy arrays.  Q/K/V are ``[B, H, n_alloc, d]`` contiguous, either
``uint16`` (bf16 bit patterns) or ``float64``; rows >= N of the token axis do not exist
for the method (they are masked, not zero keys).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sva_oracle.c")
_LIB = os.path.join(_HERE, "libsva_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no fused contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
             _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.svo_e4m3_decode.restype = C.c_double
        _lib.svo_e4m3_decode.argtypes = [C.c_uint8]
        _lib.svo_e4m3_encode.restype = C.c_uint8
        _lib.svo_e4m3_encode.argtypes = [C.c_float]
        _lib.svo_select.restype = C.c_int
        _lib.svo_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().svo_num_threads())


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _dt(a: np.ndarray) -> int:
    if a.dtype == np.float64:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError(f"oracle tensors are float64 or uint16 (bf16 bits), got {a.dtype}")


def _c(a):
    return np.ascontiguousarray(a)


def bf16_to_f64(x: np.ndarray) -> np.ndarray:
    x = _c(x)
    y = np.empty(x.shape, np.float64)
    lib().svo_bf16_to_f64(_p(x), _p(y), C.c_int64(x.size))
    return y


def e4m3_decode(code: int) -> float:
    return float(lib().svo_e4m3_decode(int(code)))


def e4m3_encode(x: float) -> int:
    return int(lib().svo_e4m3_encode(C.c_float(x)))


def quantize_e4m3(x_bf16: np.ndarray, N: int, block: int, sub: np.ndarray | None = None):
    """O10: per-(b,h,block) absmax scale, e4m3 codes. Returns (codes u8, scales f32 [B,H,Nb]).
    sub ([B,H,d] fp32, optional) is subtracted from every token in fp32 first: the K smoothing step
    of the 8-bit attention work the paper cites for its quantised attention (see k_mean)."""
    x = _c(x_bf16)
    B, H, n_alloc, d = x.shape
    Nb = -(-N // block)
    codes = np.zeros(x.shape, np.uint8)
    scales = np.zeros((B, H, Nb), np.float32)
    if sub is not None:
        sub = _c(np.asarray(sub, np.float32))
        assert sub.shape == (B, H, d)
    lib().svo_quantize_e4m3(_p(x), _p(sub), B * H, N, n_alloc, d, block, _p(codes), _p(scales))
    return codes, scales


def k_mean(k: np.ndarray, N: int) -> np.ndarray:
    """K smoothing, step 1: the mean key of each (b,h) over the N tokens that exist -> [B,H,d] float64.
    Subtracting it from every key adds the same amount, -scale*<q_i, mean>, to every logit of query i, so
    the softmax over keys -- and with it O and the kept-mass of any block set -- does not change, while
    the keys lose their common offset (which would otherwise eat the e4m3 range)."""
    kf = bf16_to_f64(k) if k.dtype == np.uint16 else np.asarray(k, np.float64)
    return kf[:, :, :N].mean(axis=2)


def lse_shift(q: np.ndarray, mean: np.ndarray, N: int, scale: float) -> np.ndarray:
    """K smoothing, step 2: what the smoothed problem's log-sum-exp is short of the original's,
    scale * <q_i, mean> -> [B,H,N] float64 (lse_original = lse_smoothed + lse_shift)."""
    qf = bf16_to_f64(q) if q.dtype == np.uint16 else np.asarray(q, np.float64)
    return scale * np.einsum("bhnd,bhd->bhn", qf[:, :, :N], np.asarray(mean, np.float64))


def dequantize_e4m3(codes: np.ndarray, scales: np.ndarray, N: int, block: int) -> np.ndarray:
    codes = _c(codes)
    scales = _c(scales.astype(np.float32))
    B, H, n_alloc, d = codes.shape
    out = np.empty(codes.shape, np.float64)
    lib().svo_dequantize_e4m3(_p(codes), _p(scales), B * H, N, n_alloc, d, block, _p(out))
    return out


def pool(x: np.ndarray, N: int, block: int) -> np.ndarray:
    """O1/O2: block means over valid tokens -> [B,H,Nb,d] float64."""
    x = _c(x)
    B, H, n_alloc, d = x.shape
    Nb = -(-N // block)
    out = np.empty((B, H, Nb, d), np.float64)
    lib().svo_pool(_p(x), _dt(x), B * H, N, n_alloc, d, block, _p(out))
    return out


def block_scores(qm: np.ndarray, km: np.ndarray, scale: float) -> np.ndarray:
    """O3: [B,H,Nb,Nb] float64."""
    qm, km = _c(qm), _c(km)
    B, H, Nb, d = qm.shape
    out = np.empty((B, H, Nb, Nb), np.float64)
    lib().svo_block_scores(_p(qm), _p(km), B * H, Nb, d, C.c_double(scale), _p(out))
    return out


@dataclass
class Selection:
    counts: np.ndarray       # [R] int32
    idx: np.ndarray          # [R, cap] int32, first counts[r] valid, ascending
    row_ptr: np.ndarray      # [R+1] int32
    col_idx: np.ndarray      # [nnz] int32
    score_gap: np.ndarray    # [R] float64
    mass_margin: np.ndarray  # [R] float64

    def kept(self, r: int) -> np.ndarray:
        return self.idx[r, : self.counts[r]]


def select(scores: np.ndarray, mode: int, k: int, tau: float = 1.0, win_t: int = -1,
           win_s: int = -1, blocks_per_frame: int = 0) -> Selection:
    """O4-O7 on a score tensor [..., Nb, Nb]. mode 0 top-k, 1 cumulative mass with cap k.
    A window is active when win_t >= 0 and win_s >= 0 and blocks_per_frame > 0."""
    s = _c(scores.astype(np.float64))
    Nb = s.shape[-1]
    R = s.size // Nb
    use_w = int(win_t >= 0 and win_s >= 0 and blocks_per_frame > 0)
    cap = Nb
    counts = np.zeros(R, np.int32)
    idx = np.full((R, cap), -1, np.int32)
    gap = np.zeros(R, np.float64)
    margin = np.zeros(R, np.float64)
    rc = lib().svo_select(_p(s), R, Nb, mode, k, C.c_double(tau), use_w, max(win_t, 0),
                          max(win_s, 0), blocks_per_frame, cap, _p(counts), _p(idx), _p(gap),
                          _p(margin))
    if rc != 0:
        raise RuntimeError("oracle select: capacity exceeded")
    row_ptr = np.zeros(R + 1, np.int32)
    lib().svo_row_ptr(_p(counts), R, _p(row_ptr))
    col = np.concatenate([idx[r, : counts[r]] for r in range(R)]) if R else np.zeros(0, np.int32)
    return Selection(counts, idx, row_ptr, _c(col.astype(np.int32)), gap, margin)


def attn_rows(q, k, v, N: int, block: int, scale: float, row_ptr, col_idx, rows=None):
    """O8: attention over the kept blocks for the listed CSR rows (all rows if None).
    Returns (o [n_rows, block, d] f64, lse [n_rows, block] f64); query tokens >= N are NaN."""
    q, k, v = _c(q), _c(k), _c(v)
    B, H, n_alloc, d = q.shape
    Nb = -(-N // block)
    row_ptr = _c(np.asarray(row_ptr, np.int32))
    col_idx = _c(np.asarray(col_idx, np.int32))
    if rows is None:
        rows_arr, n_rows = None, B * H * Nb
    else:
        rows_arr = _c(np.asarray(rows, np.int32))
        n_rows = rows_arr.size
    o = np.full((n_rows, block, d), np.nan, np.float64)
    lse = np.full((n_rows, block), np.nan, np.float64)
    lib().svo_attn_rows(_p(q), _dt(q), _p(k), _dt(k), _p(v), _dt(v), B * H, N, n_alloc, d, block,
                        C.c_double(scale), _p(row_ptr), _p(col_idx), _p(rows_arr), n_rows, _p(o),
                        _p(lse))
    return o, lse


def dense_attn_rows(q, k, v, N: int, block: int, scale: float, rows=None):
    """O9: dense attention over all valid keys, same output convention as attn_rows."""
    q, k, v = _c(q), _c(k), _c(v)
    B, H, n_alloc, d = q.shape
    Nb = -(-N // block)
    if rows is None:
        rows_arr, n_rows = None, B * H * Nb
    else:
        rows_arr = _c(np.asarray(rows, np.int32))
        n_rows = rows_arr.size
    o = np.full((n_rows, block, d), np.nan, np.float64)
    lse = np.full((n_rows, block), np.nan, np.float64)
    lib().svo_dense_attn_rows(_p(q), _dt(q), _p(k), _dt(k), _p(v), _dt(v), B * H, N, n_alloc, d,
                              block, C.c_double(scale), _p(rows_arr), n_rows, _p(o), _p(lse))
    return o, lse


def select_from_qk(q, k, N: int, block: int, scale: float, mode: int, kk: int, tau: float = 1.0,
                   win_t: int = -1, win_s: int = -1, blocks_per_frame: int = 0):
    """O1-O7 end to end. Returns (Selection, scores [B,H,Nb,Nb])."""
    s = block_scores(pool(q, N, block), pool(k, N, block), scale)
    return select(s, mode, kk, tau, win_t, win_s, blocks_per_frame), s


def gather_tokens(x: np.ndarray, token_idx: np.ndarray) -> np.ndarray:
    """Token-subset gather (the paper's token pruning keeps a subset of the tokens):
    out[b, h, m, :] = x[b, h, token_idx[b, m], :].  The definition written out, one row at a time."""
    Bq, Hq, _, d = x.shape
    M = token_idx.shape[1]
    out = np.zeros((Bq, Hq, M, d), x.dtype)
    for b in range(Bq):
        for m in range(M):
            out[b, :, m, :] = x[b, :, int(token_idx[b, m]), :]
    return out


def scatter_tokens(x: np.ndarray, token_idx: np.ndarray, dst: np.ndarray) -> np.ndarray:
    """Inverse of gather_tokens: a copy of dst with dst[b, h, token_idx[b, m], :] = x[b, h, m, :];
    the rows that token_idx does not name keep their contents."""
    out = dst.copy()
    for b in range(x.shape[0]):
        for m in range(token_idx.shape[1]):
            out[b, :, int(token_idx[b, m]), :] = x[b, :, m, :]
    return out


def qk_norm_rope(x: np.ndarray, g: np.ndarray, cos: np.ndarray, sin: np.ndarray, N: int, eps: float) -> np.ndarray:
    """The attention prologue the paper lists among its lossless fusion flags (fused QK-norm + RoPE), the two
    steps one after the other in float64, for one of Q / K.  x [B,H,n_alloc,d] (bf16 bits or float64),
    g [d], cos / sin [N, d/2].  Per token n and head:
      RMS norm over the head dimension:  u_c = x_c / sqrt(mean_c(x_c^2) + eps) * g_c
      rotary embedding on adjacent pairs: y_{2i}   = u_{2i} cos[n,i] - u_{2i+1} sin[n,i]
                                          y_{2i+1} = u_{2i+1} cos[n,i] + u_{2i} sin[n,i]
    Tokens >= N do not exist; their rows come back as zeros.  Returns float64 [B,H,n_alloc,d]."""
    xf = bf16_to_f64(x) if x.dtype == np.uint16 else np.asarray(x, np.float64)
    Bq, Hq, n_alloc, d = xf.shape
    g = np.asarray(g, np.float64)
    cos, sin = np.asarray(cos, np.float64), np.asarray(sin, np.float64)
    assert g.shape == (d,) and cos.shape == (N, d // 2) and sin.shape == (N, d // 2)
    out = np.zeros_like(xf)
    for b in range(Bq):
        for h in range(Hq):
            xs = xf[b, h, :N]
            u = xs / np.sqrt((xs * xs).mean(axis=1, keepdims=True) + eps) * g
            ue, uo = u[:, 0::2], u[:, 1::2]
            out[b, h, :N, 0::2] = ue * cos - uo * sin
            out[b, h, :N, 1::2] = uo * cos + ue * sin
    return out


from .remainder import attn_remainder_rows, block_stats, merge as merge_lse, remainder_rows  # noqa: E402,F401
