"""The C-ABI library loads without a GPU, exports what include/sva.h declares, and rejects bad
arguments on the host before any launch."""
import ctypes as C
import os
import re

import pytest

from paper_2606_23743_b200 import binding as B
from paper_2606_23743_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.lib()


def test_header_symbols_exported(lib):
    names = set()
    for header in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(sva_[a-z0-9_]+)\s*\(", text))
    assert names == set(B.EXPORTS) | set(B.DEBUG_EXPORTS), names ^ (set(B.EXPORTS) | set(B.DEBUG_EXPORTS))
    for n in names:
        assert hasattr(lib, n), n
        assert callable(getattr(B, n[len("sva_"):], None)), f"no binding function of the same name for {n}"


def _problem(**kw):
    p = B.Problem()
    p.B, p.H, p.N, p.d, p.block = 1, 2, 1024, 128, 128
    for f in ("q_stride", "k_stride", "v_stride", "o_stride"):
        setattr(p, f, (C.c_int64 * 3)(2 * 1024 * 128, 1024 * 128, 128))
    p.softmax_scale = 0.0
    p.qk_dtype = 0
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def test_status_strings(lib):
    assert B.status_string(0) == "ok"
    assert "workspace" in B.status_string(3)
    assert "unknown" in B.status_string(99)


def test_workspace_and_capacity(lib):
    p = _problem()
    s = B.make_select(0, 4)
    Nb, R = 8, 16
    assert B.select_max_nnz(p, s) == R * 4
    pooled = 2 * (2 * Nb * 128 * 4)
    scores = R * Nb * 4                                                   # the score matrix
    assert B.select_workspace_bytes(p, s) == pooled + scores             # fixed-count rows: no staging
    sm = B.make_select(1, 4, 0.9)
    assert B.select_workspace_bytes(p, sm) >= pooled + scores + R * 4 * 4 + R * 4  # staged rows + counts
    sw = B.make_select(0, 4, 1.0, 1, 1, 4)                                # 3x3 window > k
    assert B.select_max_nnz(p, sw) == R * 8                               # window clipped to Nb = 8
    assert B.select_max_nnz(p, B.make_select(0, 100)) == R * Nb          # k above Nb means Nb
    assert B.select_workspace_bytes(_problem(d=100), s) == 0


def test_rejects_bad_arguments_before_launch(lib):
    p = _problem()
    s = B.make_select(0, 4)
    one = C.c_void_p(256)      # non-null, aligned, never dereferenced: validation fails first
    vp = C.c_void_p
    def sel(p, s, q=one, k=one, rp=one, ci=one, ws=one, wsb=1 << 30):
        return lib.sva_block_select(C.byref(p), C.byref(s), q, k, None, None, rp, ci, None, ws, wsb, None)
    assert sel(_problem(d=100), s) == 2
    assert sel(_problem(block=32), s) == 2
    assert sel(_problem(N=0), s) == 1
    assert sel(p, B.make_select(0, 0)) == 1
    assert sel(p, B.make_select(2, 4)) == 1
    assert sel(p, B.make_select(1, 4, 0.0)) == 1
    assert sel(p, B.make_select(0, 4, 1.0, 1, 1, 3)) == 1            # Nb not a multiple of strips/frame
    assert sel(p, s, q=None) == 1
    assert sel(_problem(N=64 * 1025, block=64), s) == 2                # more than 1024 blocks per head
    assert sel(p, s, ws=None) == 3
    assert sel(p, s, wsb=16) == 3
    assert sel(p, s, q=vp(8)) == 5
    assert sel(p, s, ws=vp(128)) == 5
    assert sel(_problem(qk_dtype=1), s) == 1                          # fp8 without scales
    bad = _problem(); bad.q_stride = (C.c_int64 * 3)(0, 0, 132)
    assert sel(bad, s) == 5

    def att(p, q=one, k=one, v=one, o=one, rp=one, ci=one):
        return lib.sva_block_sparse_attn_fwd(C.byref(p), q, k, v, None, None, rp, ci, o, None, None, None, 0, None)
    assert att(_problem(d=96)) == 2
    assert att(p, v=None) == 1
    assert att(p, rp=None) == 1
    assert att(p, o=vp(4)) == 5
    assert att(_problem(qk_dtype=7)) == 1
    assert lib.sva_dense_attn_fwd(C.byref(p), one, one, None, None, None, one, None, None, None, 0, None) == 1
    assert B.attn_workspace_bytes(p) == 1 * 2 * 8 * 128 * 128 * 2 + 256  # transposed V tiles + row counter
    # the two-step form of the bf16 tensor-core path
    prep = lambda pp, v=one, ws=one, nb=1 << 30: lib.sva_attn_prepare_v(C.byref(pp), v, ws, nb, None)
    assert prep(p, v=None) == 1
    assert prep(p, ws=None) == 3
    assert prep(p, nb=16) == 3
    assert prep(p, ws=vp(4096 + 16)) == 5
    assert prep(_problem(d=96)) == 2
    assert prep(_problem(d=64), ws=None) == 3                             # d = 64 runs on the same kernel (padded to 128)
    att2 = lambda pp, q=one, rp=one, ci=one, ws=None, qs=None: lib.sva_block_sparse_attn_fwd_prepared(
        C.byref(pp), q, one, qs, qs, rp, ci, one, None, None, ws, 0, None)
    assert att2(p, q=None) == 1
    assert att2(p, ci=None) == 1
    assert att2(p) == 3                                                   # no workspace
    assert att2(_problem(qk_dtype=1)) == 1                                # e4m3 Q/K without their scales
    assert att2(_problem(qk_dtype=1), qs=one) == 3                        # ... with them: next complaint is the workspace
    assert B.attn_workspace_bytes(_problem(d=64)) == 1 * 2 * 8 * 128 * 128 * 2 + 256   # d = 64: V tiles padded to 128 d-rows
    assert B.attn_workspace_bytes(_problem(d=64, qk_dtype=1)) == 1 * 2 * 8 * 128 * 128 * 2 + 256
    assert B.attn_workspace_bytes(_problem(d=96)) == 0                   # unsupported shape
    # 64-token blocks: transposed V, counter, tile lists (R2 = 16 tile rows, 16 key blocks, 32 CSR rows)
    assert B.attn_workspace_bytes(_problem(block=64)) == 2 * 1024 * 128 * 2 + 256 + 256 + 256 + ((((32 * 16 + 16) // 2 + 2) * 4 + 255) // 256) * 256
    assert B.attn_workspace_bytes(_problem(qk_dtype=1)) == 1 * 2 * 8 * 128 * 128 * 2 + 256   # e4m3 Q/K: V is still bf16
    assert att(p) == 3                                                   # bf16 tensor-core path without workspace
    assert lib.sva_quantize_qk_fp8(C.byref(p), one, one, one, None, one, one, None) == 1
    bad = _problem(); bad.k_stride = (C.c_int64 * 3)(0, 0, 136)
    assert lib.sva_quantize_qk_fp8(C.byref(bad), one, one, one, one, one, one, None) == 5
    # the fused prologue: optional outputs come in whole groups
    pro = lambda pp, q=one, g=one, qo=one, qm=one, km=one, q8=None, k8=None, qs=None, ks=None, eps=1e-6: \
        lib.sva_qk_norm_rope_pool(C.byref(pp), q, one, g, one, one, one, C.c_float(eps), qo, one, qm, km, q8, k8, qs, ks, None)
    assert pro(p, q=None) == 1 and pro(p, g=None) == 1 and pro(p, qo=None) == 1
    assert pro(p, eps=-1.0) == 1
    assert pro(p, km=None) == 1                                           # one mean without the other
    assert pro(p, q8=one) == 1 and pro(p, q8=one, k8=one, qs=one) == 1    # codes without all of their scales
    assert pro(p, q=vp(264)) == 5
    assert pro(bad, q8=one, k8=one, qs=one, ks=one) == 5                  # stride 136 is fine for bf16, not for the codes
    # pooling alone
    pool = lambda pp, q=one, qm=one: lib.sva_pool_qk(C.byref(pp), q, one, None, None, qm, one, None)
    assert pool(p, q=None) == 1 and pool(p, qm=None) == 1 and pool(p, qm=vp(260)) == 5
    assert pool(_problem(qk_dtype=1)) == 1                                # e4m3 codes without their scales
    # routing from given means
    selp = lambda pp, ss, qm=one, km=one, rp=one, ci=one, ws=one, wsb=1 << 30: \
        lib.sva_block_select_pooled(C.byref(pp), C.byref(ss), qm, km, rp, ci, None, ws, C.c_size_t(wsb), None)
    assert selp(p, s, qm=None) == 1 and selp(p, s, ci=None) == 1
    assert selp(p, s, ws=None) == 3 and selp(p, s, wsb=16) == 3
    assert selp(p, s, qm=vp(260)) == 5
    assert selp(p, B.make_select(0, 0)) == 1
    # the smoothing quantiser: k_mean and its workspace are required, the lse shift is optional
    sm = lambda pp, mean=one, ws=one, nb=1 << 30: lib.sva_quantize_qk_fp8_smooth_k(
        C.byref(pp), one, one, one, one, one, one, mean, None, ws, C.c_size_t(nb), None)
    assert B.smooth_workspace_bytes(p) == 4 * 1 * 2 * 8 * 128
    assert sm(p, mean=None) == 1
    assert sm(p, ws=None) == 3 and sm(p, nb=B.smooth_workspace_bytes(p) - 1) == 3
    assert sm(p, ws=vp(4096 + 8)) == 5
    assert sm(bad) == 5


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", "/nonexistent/libsva.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()


def test_token_move_rejects_bad_arguments_before_launch(lib):
    one = C.c_void_p(256)
    st3 = (C.c_int64 * 3)(2 * 1024 * 128, 1024 * 128, 128)
    def mv(fn, src=one, idx=one, dst=one, B_=1, H=2, M=512, n=1024, d=128, eb=2, ss=st3, sd=st3):
        return fn(src, ss, idx, B_, H, M, n, d, eb, dst, sd, None, None)
    for fn in (lib.sva_gather_tokens, lib.sva_scatter_tokens):
        assert mv(fn, src=None) == 1
        assert mv(fn, idx=None) == 1
        assert mv(fn, M=2048) == 1                       # more kept tokens than tokens
        assert mv(fn, eb=3) == 1
        assert mv(fn, d=100) == 2                        # rows must be whole 16-byte vectors
        assert mv(fn, dst=C.c_void_p(8)) == 5
        assert mv(fn, ss=(C.c_int64 * 3)(0, 0, 132)) == 5
        assert mv(fn, ss=(C.c_int64 * 3)(0, 0, 64)) == 1  # row stride shorter than a row


def test_routing_limits_are_refused_on_the_host(lib):
    """More than 1024 blocks per head, or a CSR capacity R * cap beyond int32: size queries answer 0 and the
    routing calls return UNSUPPORTED before any launch (no silent wrap of the int32 offsets)."""
    big_nb = _problem(N=128 * 1025)                       # Nb = 1025
    s = B.make_select(0, 4)
    assert B.select_max_nnz(big_nb, s) == 0 and B.select_workspace_bytes(big_nb, s) == 0
    many = _problem(B=32, H=512, N=128 * 1024)            # R = 2^24 rows, k = 128 -> 2^31 entries
    s64 = B.make_select(0, 128)
    assert B.select_max_nnz(many, s64) == 0 and B.select_workspace_bytes(many, s64) == 0
    assert B.select_max_nnz(many, B.make_select(0, 127)) == (32 * 512 * 1024) * 127
    fake = C.c_void_p(256)
    for p, sel in ((big_nb, s), (many, s64)):
        for fn, args in ((lib.sva_block_select, (fake, fake, None, None, fake, fake, None, fake, C.c_size_t(1 << 40), None)),
                         (lib.sva_block_select_pooled, (fake, fake, fake, fake, None, fake, C.c_size_t(1 << 40), None)),
                         (lib.sva_block_select_noalloc, (fake, fake, None, None, fake, fake, None, None))):
            assert fn(C.byref(p), C.byref(sel), *args) == 2, fn
