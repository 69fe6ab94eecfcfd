"""Thin ctypes binding over the C ABI declared in include/sva.h.

Argument marshalling only: every step of the path runs in the CUDA kernels.  torch is used
for device memory and streams.  There is no CPU fallback: a missing library raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsva.so")
_lib = None

SVA_OK = 0
SVA_BF16, SVA_FP8_E4M3 = 0, 1
SVA_DEV_BAD_INDEX, SVA_DEV_TIMEOUT = 1, 2

EXPORTS = [
    "sva_select_max_nnz", "sva_select_workspace_bytes", "sva_block_select",
    "sva_block_sparse_attn_fwd", "sva_dense_attn_fwd", "sva_block_sparse_attn_fwd_simt",
    "sva_quantize_qk_fp8", "sva_status_string", "sva_block_select_noalloc", "sva_attn_workspace_bytes",
    "sva_attn_prepare_v", "sva_block_sparse_attn_fwd_prepared", "sva_gather_tokens", "sva_scatter_tokens",
    "sva_attn_one_call_workspace_bytes", "sva_quantize_qk_fp4", "sva_block_sparse_attn_fwd_fp4", "sva_attn_remainder_workspace_bytes", "sva_block_sparse_attn_remainder_fwd", "sva_smooth_workspace_bytes", "sva_quantize_qk_fp8_smooth_k", "sva_block_select_pooled", "sva_qk_norm_rope_pool", "sva_pool_qk",
]
DEBUG_EXPORTS = ["sva_debug_set_prof_buffer", "sva_debug_set_mode", "sva_debug_set_wait_limit"]
NOALLOC_SCRATCH_BYTES = 16 << 20


class Problem(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("N", C.c_int32), ("d", C.c_int32),
                ("block", C.c_int32),
                ("q_stride", C.c_int64 * 3), ("k_stride", C.c_int64 * 3),
                ("v_stride", C.c_int64 * 3), ("o_stride", C.c_int64 * 3),
                ("softmax_scale", C.c_float), ("qk_dtype", C.c_int32)]


class Select(C.Structure):
    _fields_ = [("mode", C.c_int32), ("k", C.c_int32), ("mass", C.c_float),
                ("win_t", C.c_int32), ("win_s", C.c_int32), ("blocks_per_frame", C.c_int32)]


class SvaError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


def lib():
    """Loads libsva.so (built in-tree by paper_2606_23743_b200.build). Raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2606_23743_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(_LIB_PATH)
        vp = C.c_void_p
        L.sva_select_max_nnz.restype = C.c_int64
        L.sva_select_max_nnz.argtypes = [C.POINTER(Problem), C.POINTER(Select)]
        L.sva_select_workspace_bytes.restype = C.c_size_t
        L.sva_select_workspace_bytes.argtypes = [C.POINTER(Problem), C.POINTER(Select)]
        L.sva_block_select.restype = C.c_int
        L.sva_block_select.argtypes = [C.POINTER(Problem), C.POINTER(Select), vp, vp, vp, vp, vp, vp,
                                       vp, vp, C.c_size_t, vp]
        L.sva_block_select_noalloc.restype = C.c_int
        L.sva_block_select_noalloc.argtypes = [C.POINTER(Problem), C.POINTER(Select), vp, vp, vp, vp, vp, vp,
                                               vp, vp]
        L.sva_attn_one_call_workspace_bytes.restype = C.c_size_t
        L.sva_attn_one_call_workspace_bytes.argtypes = [C.POINTER(Problem)]
        L.sva_attn_workspace_bytes.restype = C.c_size_t
        L.sva_attn_workspace_bytes.argtypes = [C.POINTER(Problem)]
        L.sva_block_sparse_attn_fwd.restype = C.c_int
        L.sva_block_sparse_attn_fwd.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                                C.c_size_t, vp]
        L.sva_block_sparse_attn_fwd_simt.restype = C.c_int
        L.sva_block_sparse_attn_fwd_simt.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.sva_dense_attn_fwd.restype = C.c_int
        L.sva_dense_attn_fwd.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        L.sva_attn_remainder_workspace_bytes.restype = C.c_size_t
        L.sva_attn_remainder_workspace_bytes.argtypes = [C.POINTER(Problem), C.c_int32]
        L.sva_block_sparse_attn_remainder_fwd.restype = C.c_int
        L.sva_block_sparse_attn_remainder_fwd.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_int32, vp,
                                                          C.c_size_t, vp]
        L.sva_attn_prepare_v.restype = C.c_int
        L.sva_attn_prepare_v.argtypes = [C.POINTER(Problem), vp, vp, C.c_size_t, vp]
        L.sva_block_sparse_attn_fwd_prepared.restype = C.c_int
        L.sva_block_sparse_attn_fwd_prepared.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        for fn in (L.sva_gather_tokens, L.sva_scatter_tokens):
            fn.restype = C.c_int
            fn.argtypes = [vp, C.POINTER(C.c_int64), vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                           C.c_int32, vp, C.POINTER(C.c_int64), vp, vp]
        L.sva_quantize_qk_fp8.restype = C.c_int
        L.sva_quantize_qk_fp8.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp]
        L.sva_quantize_qk_fp4.restype = C.c_int
        L.sva_quantize_qk_fp4.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        L.sva_block_sparse_attn_fwd_fp4.restype = C.c_int
        L.sva_block_sparse_attn_fwd_fp4.argtypes = [C.POINTER(Problem)] + [vp] * 13 + [C.c_size_t, vp]
        L.sva_smooth_workspace_bytes.restype = C.c_size_t
        L.sva_smooth_workspace_bytes.argtypes = [C.POINTER(Problem)]
        L.sva_quantize_qk_fp8_smooth_k.restype = C.c_int
        L.sva_quantize_qk_fp8_smooth_k.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        L.sva_pool_qk.restype = C.c_int
        L.sva_pool_qk.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, vp]
        L.sva_block_select_pooled.restype = C.c_int
        L.sva_block_select_pooled.argtypes = [C.POINTER(Problem), C.POINTER(Select), vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        L.sva_qk_norm_rope_pool.restype = C.c_int
        L.sva_qk_norm_rope_pool.argtypes = [C.POINTER(Problem), vp, vp, vp, vp, vp, vp, C.c_float, vp, vp, vp, vp, vp, vp,
                                            vp, vp, vp]
        # test and tuning aids (include/sva_debug.h): process-global settings
        L.sva_debug_set_prof_buffer.restype = None
        L.sva_debug_set_prof_buffer.argtypes = [vp]
        L.sva_debug_set_mode.restype = None
        L.sva_debug_set_mode.argtypes = [C.c_int]
        L.sva_debug_set_wait_limit.restype = C.c_int
        L.sva_debug_set_wait_limit.argtypes = [C.c_longlong]
        L.sva_status_string.restype = C.c_char_p
        L.sva_status_string.argtypes = [C.c_int]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().sva_status_string(int(status)).decode()


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _strides(t):
    assert t.dim() == 4 and t.stride(3) == 1, "tensors are [B,H,N,d] with d contiguous"
    return (C.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


def make_problem(q, k, v, o, N: int, block: int, scale: float = 0.0, fp8: bool = False) -> Problem:
    """q,k,v,o: [B,H,n_alloc,d] device tensors (d contiguous); N = valid tokens <= n_alloc."""
    B, H, _, d = q.shape
    p = Problem()
    p.B, p.H, p.N, p.d, p.block = B, H, N, d, block
    p.q_stride, p.k_stride = _strides(q), _strides(k)
    p.v_stride = _strides(v) if v is not None else _strides(q)
    p.o_stride = _strides(o) if o is not None else _strides(q)
    p.softmax_scale = scale
    p.qk_dtype = SVA_FP8_E4M3 if fp8 else SVA_BF16
    return p


def make_select(mode: int, k: int, mass: float = 1.0, win_t: int = -1, win_s: int = -1,
                blocks_per_frame: int = 0) -> Select:
    return Select(mode, k, mass, win_t, win_s, blocks_per_frame)


def select_max_nnz(p: Problem, s: Select) -> int:
    return int(lib().sva_select_max_nnz(C.byref(p), C.byref(s)))


def select_workspace_bytes(p: Problem, s: Select) -> int:
    return int(lib().sva_select_workspace_bytes(C.byref(p), C.byref(s)))


def block_select(p: Problem, s: Select, q, k, row_ptr, col_idx, workspace, q_scale=None, k_scale=None,
                 block_scores=None) -> None:
    rc = lib().sva_block_select(C.byref(p), C.byref(s), _ptr(q), _ptr(k), _ptr(q_scale), _ptr(k_scale),
                                _ptr(row_ptr), _ptr(col_idx), _ptr(block_scores), _ptr(workspace),
                                workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_block_select")


def block_select_noalloc(p: Problem, s: Select, q, k, row_ptr, col_idx, q_scale=None, k_scale=None,
                         block_scores=None) -> None:
    """sva_block_select for callers that cannot allocate: the scratch is the library's built-in
    device array (NOALLOC_SCRATCH_BYTES); raises SvaError(status 6) when the problem needs more.
    Calls share that array, so calls that could overlap on the GPU must be serialised."""
    rc = lib().sva_block_select_noalloc(C.byref(p), C.byref(s), _ptr(q), _ptr(k), _ptr(q_scale),
                                        _ptr(k_scale), _ptr(row_ptr), _ptr(col_idx), _ptr(block_scores),
                                        _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_block_select_noalloc")


def attn_workspace_bytes(p: Problem) -> int:
    return int(lib().sva_attn_workspace_bytes(C.byref(p)))


def _ws_bytes(ws):
    return ws.numel() * ws.element_size() if ws is not None else 0


def block_sparse_attn_fwd_simt(p: Problem, q, k, v, row_ptr, col_idx, o, lse=None, status=None, q_scale=None,
                               k_scale=None) -> None:
    """The diagnostic CUDA-core twin (row_ptr None = dense)."""
    rc = lib().sva_block_sparse_attn_fwd_simt(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(q_scale),
                                              _ptr(k_scale), _ptr(row_ptr), _ptr(col_idx), _ptr(o),
                                              _ptr(lse), _ptr(status), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_block_sparse_attn_fwd_simt")


def block_sparse_attn_fwd(p: Problem, q, k, v, row_ptr, col_idx, o, lse=None, status=None, q_scale=None,
                          k_scale=None, simt: bool = False, workspace=None) -> None:
    if simt:
        return block_sparse_attn_fwd_simt(p, q, k, v, row_ptr, col_idx, o, lse, status, q_scale, k_scale)
    rc = lib().sva_block_sparse_attn_fwd(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(q_scale),
                                         _ptr(k_scale), _ptr(row_ptr), _ptr(col_idx), _ptr(o), _ptr(lse),
                                         _ptr(status), _ptr(workspace), _ws_bytes(workspace), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_block_sparse_attn_fwd")


def dense_attn_fwd(p: Problem, q, k, v, o, lse=None, status=None, q_scale=None, k_scale=None,
                   workspace=None) -> None:
    rc = lib().sva_dense_attn_fwd(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(q_scale), _ptr(k_scale),
                                  _ptr(o), _ptr(lse), _ptr(status), _ptr(workspace), _ws_bytes(workspace),
                                  _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_dense_attn_fwd")


def attn_prepare_v(p: Problem, v, workspace) -> None:
    """First half of the bf16 tensor-core path: V -> tiled transposed copy in `workspace` (on the current stream)."""
    rc = lib().sva_attn_prepare_v(C.byref(p), _ptr(v), _ptr(workspace), _ws_bytes(workspace), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_attn_prepare_v")


def block_sparse_attn_fwd_prepared(p: Problem, q, k, row_ptr, col_idx, o, lse=None, status=None,
                                   workspace=None, q_scale=None, k_scale=None) -> None:
    """Second half: the attention kernel alone on a workspace that attn_prepare_v filled (row_ptr None = dense)."""
    rc = lib().sva_block_sparse_attn_fwd_prepared(C.byref(p), _ptr(q), _ptr(k), _ptr(q_scale), _ptr(k_scale),
                                                  _ptr(row_ptr), _ptr(col_idx), _ptr(o), _ptr(lse), _ptr(status),
                                                  _ptr(workspace), _ws_bytes(workspace), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_block_sparse_attn_fwd_prepared")


def _token_move(name, src, token_idx, dst, status):
    Bq, Hq, n_src, d = src.shape
    M = token_idx.shape[1]
    n_full = dst.shape[2] if name == "sva_scatter_tokens" else n_src
    rc = getattr(lib(), name)(_ptr(src), _strides(src), _ptr(token_idx), Bq, Hq, M, n_full, d, src.element_size(),
                              _ptr(dst), _strides(dst), _ptr(status), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, name)


def gather_tokens(src, token_idx, dst, status=None) -> None:
    """dst[b,h,m,:] = src[b,h,token_idx[b,m],:]; src [B,H,N,d], token_idx [B,M] int32, dst [B,H,>=M,d]."""
    _token_move("sva_gather_tokens", src, token_idx, dst, status)


def scatter_tokens(src, token_idx, dst, status=None) -> None:
    """dst[b,h,token_idx[b,m],:] = src[b,h,m,:]; the other rows of dst keep their contents."""
    _token_move("sva_scatter_tokens", src, token_idx, dst, status)


def quantize_qk_fp8(p: Problem, q, k, q8, k8, q_scale, k_scale) -> None:
    rc = lib().sva_quantize_qk_fp8(C.byref(p), _ptr(q), _ptr(k), _ptr(q8), _ptr(k8), _ptr(q_scale),
                                   _ptr(k_scale), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_quantize_qk_fp8")


def smooth_workspace_bytes(p: Problem) -> int:
    return int(lib().sva_smooth_workspace_bytes(C.byref(p)))


def quantize_qk_fp8_smooth_k(p: Problem, q, k, q8, k8, q_scale, k_scale, k_mean, lse_shift, workspace) -> None:
    rc = lib().sva_quantize_qk_fp8_smooth_k(C.byref(p), _ptr(q), _ptr(k), _ptr(q8), _ptr(k8), _ptr(q_scale),
                                            _ptr(k_scale), _ptr(k_mean), _ptr(lse_shift), _ptr(workspace),
                                            C.c_size_t(_ws_bytes(workspace)), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_quantize_qk_fp8_smooth_k")


def block_select_pooled(p: Problem, s: Select, q_mean, k_mean, row_ptr, col_idx, workspace, block_scores=None) -> None:
    rc = lib().sva_block_select_pooled(C.byref(p), C.byref(s), _ptr(q_mean), _ptr(k_mean), _ptr(row_ptr), _ptr(col_idx),
                                       _ptr(block_scores), _ptr(workspace), C.c_size_t(_ws_bytes(workspace)), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_block_select_pooled")


def qk_norm_rope_pool(p: Problem, q, k, g_q, g_k, cos_table, sin_table, eps, q_out, k_out, q_mean=None, k_mean=None,
                      q8=None, k8=None, q_scale=None, k_scale=None) -> None:
    rc = lib().sva_qk_norm_rope_pool(C.byref(p), _ptr(q), _ptr(k), _ptr(g_q), _ptr(g_k), _ptr(cos_table),
                                     _ptr(sin_table), C.c_float(eps), _ptr(q_out), _ptr(k_out), _ptr(q_mean),
                                     _ptr(k_mean), _ptr(q8), _ptr(k8), _ptr(q_scale), _ptr(k_scale), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_qk_norm_rope_pool")


def pool_qk(p: Problem, q, k, q_mean, k_mean, q_scale=None, k_scale=None) -> None:
    rc = lib().sva_pool_qk(C.byref(p), _ptr(q), _ptr(k), _ptr(q_scale), _ptr(k_scale), _ptr(q_mean), _ptr(k_mean),
                           _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_pool_qk")


def debug_set_prof_buffer(buf) -> None:
    """Cycle counter of the attention kernel (include/sva_debug.h): a zeroed device int64 tensor of >= 320
    entries, entry 319 receives the cycle count of the longest CTA of later launches; None switches it off."""
    lib().sva_debug_set_prof_buffer(_ptr(buf))


def debug_set_mode(bits: int) -> None:
    """Kernel behaviour switches of later attention launches (include/sva_debug.h); 0 = normal."""
    lib().sva_debug_set_mode(int(bits))


def debug_set_wait_limit(cycles: int) -> None:
    """SM cycles a device-side wait may last before its CTA gives up; <= 0 restores the default."""
    if lib().sva_debug_set_wait_limit(C.c_longlong(int(cycles))) != 0:
        raise RuntimeError("sva_debug_set_wait_limit failed")


def attn_remainder_workspace_bytes(p: Problem, order: int = 0) -> int:
    return int(lib().sva_attn_remainder_workspace_bytes(C.byref(p), int(order)))


def block_sparse_attn_remainder_fwd(p: Problem, q, k, v, row_ptr, col_idx, o, lse=None, status=None, order: int = 0,
                                    workspace=None, block_scores=None) -> None:
    """Exact attention over the kept blocks plus the approximate remainder of the dropped ones (order 0: block means;
    order 1: plus the first-order term, which needs the routing's score matrix)."""
    rc = lib().sva_block_sparse_attn_remainder_fwd(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(row_ptr), _ptr(col_idx),
                                                   _ptr(block_scores), _ptr(o), _ptr(lse), _ptr(status), int(order),
                                                   _ptr(workspace), _ws_bytes(workspace), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_block_sparse_attn_remainder_fwd")


def quantize_qk_fp4(p: Problem, q, k, q4, k4, q_sf, k_sf, q_g, k_g, workspace) -> None:
    """Block-scaled 4-bit codes, e4m3 block scales (MMA tile order) and per-(b,h) fp32 scales of Q and K."""
    rc = lib().sva_quantize_qk_fp4(C.byref(p), _ptr(q), _ptr(k), _ptr(q4), _ptr(k4), _ptr(q_sf), _ptr(k_sf), _ptr(q_g),
                                   _ptr(k_g), _ptr(workspace), _ws_bytes(workspace), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_quantize_qk_fp4")


def block_sparse_attn_fwd_fp4(p: Problem, q4, k4, q_sf, k_sf, q_g, k_g, v, row_ptr, col_idx, o, lse=None, status=None,
                              workspace=None) -> None:
    """Attention over 4-bit block-scaled Q and K (row_ptr None = dense)."""
    rc = lib().sva_block_sparse_attn_fwd_fp4(C.byref(p), _ptr(q4), _ptr(k4), _ptr(q_sf), _ptr(k_sf), _ptr(q_g), _ptr(k_g),
                                             _ptr(v), _ptr(row_ptr), _ptr(col_idx), _ptr(o), _ptr(lse), _ptr(status),
                                             _ptr(workspace), _ws_bytes(workspace), _stream())
    if rc != SVA_OK:
        raise SvaError(rc, "sva_block_sparse_attn_fwd_fp4")


def attn_one_call_workspace_bytes(p: Problem) -> int:
    """Workspace the one-call attention entry points need (e4m3 Q/K: just the row counters and tile lists)."""
    return int(lib().sva_attn_one_call_workspace_bytes(C.byref(p)))
