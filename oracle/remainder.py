"""fp64 CPU oracle of the approximate remainder for dropped key blocks -- TEST INFRASTRUCTURE.

The paper's sparse-attention section describes piecewise sparse attention: the critical key blocks of a
query block are computed exactly, the non-critical ones are "compensated with first-order Taylor
approximation", and its LTX-2.3 deployment runs with the "approximate remainder enabled".  The paper prints no
formula.  The reading implemented here (parity unpinned by the paper; every step below is this build's):

  For a dropped key block J with n_J existing keys, mean key kbar_J, mean value vbar_J, expand
  exp(scale <q_i, k_j>) to first order in the deviation of the key from its block mean,
      exp(scale <q_i, k_j>)  ~=  exp(a_iJ) * (1 + scale <q_i, k_j - kbar_J>),     a_iJ = scale <q_i, kbar_J>.
  Summed over the block the first-order term of the DENOMINATOR vanishes (deviations from a mean sum to 0):
      sum_j exp(s_ij)      ~=  n_J exp(a_iJ)
      sum_j exp(s_ij) v_j  ~=  exp(a_iJ) * (n_J vbar_J + scale C_J^T q_i),     C_J = sum_j (k_j - kbar_J) v_j^T  (d x d).
  order 0 keeps only n_J exp(a_iJ) and n_J exp(a_iJ) vbar_J (the block-mean term).
  order 1 adds the C_J term.  So that the dropped blocks collapse into ONE d x d matrix per query block
  (instead of one d x d product per query and dropped block) its weight exp(a_iJ) is taken at the query
  block's mean query, exp(sbar_IJ) with sbar_IJ = scale <qbar_I, kbar_J> (the routing score): the two differ
  by scale <q_i - qbar_I, kbar_J>, a first-order quantity that multiplies a first-order term, so the change
  is of second order, like everything else that is dropped.  `order1_weight="query"` evaluates the
  uncollapsed form for comparison.

  The exact part (kept blocks) and the remainder are merged through the log-sum-exp:
      Z_i = exp(lse_exact_i) + Z_rem_i,   o_i = (exp(lse_exact_i) o_exact_i + N_rem_i) / Z_i,   lse_i = ln Z_i.
  A query block that drops nothing has no remainder and returns the exact result unchanged.

Block statistics may be rounded to bf16 (`stats="bf16"`: what a tensor-core implementation feeds its MMAs);
`stats="f64"` keeps them exact (used by the pins).

Only tests, the smoke check and the bench's CPU legs may import this module.
"""
from __future__ import annotations

import numpy as np


def _to_f64(x):
    from . import bf16_to_f64
    return bf16_to_f64(x) if x.dtype == np.uint16 else np.asarray(x, np.float64)


def _round_bf16(x: np.ndarray) -> np.ndarray:
    """fp64 -> fp32 (round to nearest) -> bf16 (round to nearest even), returned as fp64."""
    f = np.ascontiguousarray(x, np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(x.shape)


def block_stats(k, v, N: int, block: int, want_cov: bool = True):
    """Per (b, h, J): n_J, mean key, mean value and C_J = sum_j (k_j - kbar_J) v_j^T over the existing
    tokens of block J.  Returns (n [Nb], kbar [B,H,Nb,d], vbar [B,H,Nb,d], C [B,H,Nb,d,d] or None), fp64."""
    kf, vf = _to_f64(k), _to_f64(v)
    B, H, _, d = kf.shape
    Nb = -(-N // block)
    n = np.array([min(block, N - J * block) for J in range(Nb)], np.float64)
    kbar = np.zeros((B, H, Nb, d)); vbar = np.zeros((B, H, Nb, d))
    C = np.zeros((B, H, Nb, d, d)) if want_cov else None
    for b in range(B):
        for h in range(H):
            for J in range(Nb):
                lo, hi = J * block, min((J + 1) * block, N)
                kk, vv = kf[b, h, lo:hi], vf[b, h, lo:hi]
                kbar[b, h, J] = kk.sum(axis=0) / (hi - lo)
                vbar[b, h, J] = vv.sum(axis=0) / (hi - lo)
                if want_cov:
                    C[b, h, J] = (kk - kbar[b, h, J]).T @ vv
    return n, kbar, vbar, C


def remainder_rows(q, k, v, N: int, block: int, scale: float, row_ptr, col_idx, rows, order: int = 1,
                   stats: str = "f64", order1_weight: str = "block"):
    """The remainder of the listed CSR rows (query blocks) alone: (N_rem [n_rows, block, d],
    lnZ_rem [n_rows, block]) with N_rem scaled by exp(-lnZ_rem), i.e. the remainder's own normalised
    output and log-mass; rows without dropped blocks give lnZ_rem = -inf and zeros.  Absent queries NaN."""
    assert order in (0, 1) and stats in ("f64", "bf16") and order1_weight in ("block", "query")
    qf = _to_f64(q)
    B, H, _, d = qf.shape
    Nb = -(-N // block)
    n, kbar, vbar, C = block_stats(k, v, N, block, want_cov=order == 1)
    # the mean query of every block (weights of the collapsed first-order term)
    _, qbar, _, _ = block_stats(q, q, N, block, want_cov=False)
    if stats == "bf16":
        kbar, vbar = _round_bf16(kbar), _round_bf16(vbar)
        if C is not None:
            C = _round_bf16(C)
    row_ptr = np.asarray(row_ptr); col_idx = np.asarray(col_idx)
    o = np.full((len(rows), block, d), np.nan); lnz = np.full((len(rows), block), np.nan)
    for t, r in enumerate(rows):
        bh, I = divmod(int(r), Nb)
        b, h = divmod(bh, H)
        lo, hi = I * block, min((I + 1) * block, N)
        dropped = np.ones(Nb, bool)
        dropped[col_idx[row_ptr[r]:row_ptr[r + 1]]] = False
        if not dropped.any():
            o[t, : hi - lo] = 0.0
            lnz[t, : hi - lo] = -np.inf
            continue
        Jd = np.nonzero(dropped)[0]
        qi = qf[b, h, lo:hi]                                   # [nq, d]
        a = scale * qi @ kbar[b, h, Jd].T                      # [nq, |D|]
        m = a.max(axis=1, keepdims=True)
        w0 = np.exp(a - m) * n[Jd][None, :]                    # n_J exp(a_iJ - m_i)
        Z = w0.sum(axis=1)                                     # relative to m
        Nn = w0 @ vbar[b, h, Jd]
        if order == 1:
            if order1_weight == "block":
                sb = scale * (kbar[b, h, Jd] @ qbar[b, h, I])  # [|D|]
                A = np.einsum("J,Jcd->cd", np.exp(sb - sb.max()), C[b, h, Jd])       # one d x d matrix per query block
                Nn = Nn + scale * np.exp(sb.max() - m) * (qi @ A)
            else:
                Nn = Nn + scale * np.einsum("iJ,Jcd,ic->id", np.exp(a - m), C[b, h, Jd], qi)
        o[t, : hi - lo] = Nn / Z[:, None]
        lnz[t, : hi - lo] = m[:, 0] + np.log(Z)
    return o, lnz


def merge(o_exact, lse_exact, o_rem, lnz_rem):
    """Exact part and remainder merged through the log-sum-exp (both parts normalised by their own mass).
    Where the remainder is empty (lnz_rem = -inf) the exact result is returned unchanged, bit for bit."""
    o_exact, lse_exact = np.asarray(o_exact, np.float64), np.asarray(lse_exact, np.float64)
    none = np.isneginf(lnz_rem)
    empty = np.isneginf(lse_exact)                 # nothing kept: the exact part is 0/0 there and has no weight
    o_exact = np.where(empty[..., None], 0.0, o_exact)
    with np.errstate(invalid="ignore"):            # (absent queries carry NaN through)
        lse = np.logaddexp(lse_exact, lnz_rem)
        we, wr = np.exp(lse_exact - lse), np.exp(lnz_rem - lse)
        o = we[..., None] * o_exact + wr[..., None] * o_rem
    o = np.where(none[..., None], o_exact, o)
    lse = np.where(none, lse_exact, lse)
    return o, lse


def attn_remainder_rows(q, k, v, N: int, block: int, scale: float, row_ptr, col_idx, rows, order: int = 1,
                        stats: str = "f64", order1_weight: str = "block"):
    """Piecewise attention of the listed rows: exact over the kept blocks (the plain definition, the C
    oracle's attn_rows), Taylor remainder over the dropped ones, merged through the LSE.
    Returns (o [n_rows, block, d], lse [n_rows, block]); absent queries NaN."""
    from . import attn_rows
    rows = [int(r) for r in rows]
    o_e, lse_e = attn_rows(q, k, v, N, block, scale, row_ptr, col_idx, rows=rows)
    o_r, lnz_r = remainder_rows(q, k, v, N, block, scale, row_ptr, col_idx, rows, order, stats, order1_weight)
    return merge(o_e, lse_e, o_r, lnz_r)
