"""Pins for the oracle's pooling, block scores and selection (O1-O7)."""
import math

import numpy as np
import pytest

import oracle


def _block_const(vals, block, n_valid=None):
    """[Nb, d] -> [1,1,Nb*block,d] where every token of block I equals vals[I]."""
    x = np.repeat(np.asarray(vals, np.float64), block, axis=0)[None, None]
    return np.ascontiguousarray(x)


def test_pool_ragged_tail_and_garbage():
    N, block, d = 150, 64, 3
    x = np.random.default_rng(0).standard_normal((1, 2, 192, d))
    x[:, :, N:] = 1e6                                     # absent tokens must not be read
    m = oracle.pool(x, N, block)
    assert m.shape == (1, 2, 3, d)
    np.testing.assert_allclose(m[0, 1, 0], x[0, 1, :64].mean(0), rtol=1e-13)
    np.testing.assert_allclose(m[0, 1, 2], x[0, 1, 128:150].mean(0), rtol=1e-13)   # 22 valid tokens


def test_scores_integer_closed_form_and_scale():
    block = 4
    u = np.array([[1, 0, 2], [0, 3, 0], [-1, 1, 1]], float)
    w = np.array([[2, 1, 0], [1, 1, 1], [0, 0, -3]], float)
    q, k = _block_const(u, block), _block_const(w, block)
    s = oracle.block_scores(oracle.pool(q, 12, block), oracle.pool(k, 12, block), 0.5)
    np.testing.assert_array_equal(s[0, 0], 0.5 * (u @ w.T))     # exact small integers / halves
    assert s[0, 0, 0, 2] == -3.0 and s[0, 0, 2, 0] == -0.5       # not transposed


def test_topk_exact_ties_lower_index():
    # hand-written rows, including exact ties and signed zeros
    s = np.array([[[
        [5, 5, 5, 5, 5, 5],          # all tied -> 0,1,2
        [1, 9, 9, 2, 9, 9],          # four tied at 9 -> 1,2,4
        [0.0, -0.0, -1, 0.0, -2, -3],  # +0 == -0 -> 0,1,3
        [1, 2, 3, 4, 5, 6],          # -> 3,4,5
        [6, 5, 4, 3, 2, 1],          # -> 0,1,2
        [3, 1, 3, 1, 3, 1],          # -> 0,2,4
    ]]], float)
    sel = oracle.select(s, 0, 3)
    exp = [[0, 1, 2], [1, 2, 4], [0, 1, 3], [3, 4, 5], [0, 1, 2], [0, 2, 4]]
    assert [sel.kept(r).tolist() for r in range(6)] == exp
    assert sel.counts.tolist() == [3] * 6
    # gaps: tied boundary -> 0; row 3: 4 - 3 = 1
    assert sel.score_gap[0] == 0.0 and sel.score_gap[1] == 0.0 and sel.score_gap[3] == 1.0
    # k >= Nb keeps everything
    assert oracle.select(s, 0, 10).counts.tolist() == [6] * 6


def test_topk_brute_force_random():
    rng = np.random.default_rng(3)
    for Nb, k in [(16, 4), (37, 9), (64, 16), (5, 5)]:
        s = rng.integers(-3, 4, size=(2, 3, Nb, Nb)).astype(float)    # many exact ties
        sel = oracle.select(s, 0, k)
        flat = s.reshape(-1, Nb)
        for r in range(flat.shape[0]):
            order = sorted(range(Nb), key=lambda j: (-flat[r, j], j))
            assert sel.kept(r).tolist() == sorted(order[:k])
        # CSR invariants
        assert sel.row_ptr[0] == 0 and sel.row_ptr[-1] == sel.col_idx.size == flat.shape[0] * k
        assert (np.diff(sel.row_ptr) == sel.counts).all()
        for r in range(flat.shape[0]):
            seg = sel.col_idx[sel.row_ptr[r]:sel.row_ptr[r + 1]]
            assert (np.diff(seg) > 0).all() and seg.min() >= 0 and seg.max() < Nb


@pytest.mark.parametrize("Nb,m,a,tau", [(32, 6, 4.0, 0.5), (32, 6, 4.0, 0.9), (64, 10, 3.0, 0.8),
                                        (16, 3, 8.0, 0.99), (20, 5, 2.0, 0.3)])
def test_mass_rule_two_level_closed_form(Nb, m, a, tau):
    """m blocks at score a, the rest at 0: n = ceil(tau * Z / e^a) while that is <= m."""
    row = np.zeros(Nb)
    hi = np.arange(Nb - m, Nb)                 # put the high blocks at the END of the row
    row[hi] = a
    Z = m * math.exp(a) + (Nb - m)
    n_hi = math.ceil(tau * Z / math.exp(a) - 1e-12)
    if n_hi <= m:
        n = n_hi
        exp_set = hi[:n].tolist()              # ties among the high blocks -> lower index first
    else:
        n = m + math.ceil((tau * Z - m * math.exp(a)) - 1e-12)
        exp_set = sorted(hi.tolist() + list(range(n - m)))
    s = np.tile(row, (1, 1, 2, 1))
    sel = oracle.select(s, 1, Nb, tau)
    assert sel.counts.tolist() == [n, n]
    assert sel.kept(0).tolist() == exp_set
    # the cap and the floor of one block
    assert oracle.select(s, 1, 2, tau).counts.tolist() == [min(n, 2)] * 2
    assert oracle.select(s, 1, Nb, 1e-9).counts.tolist() == [1, 1]
    assert oracle.select(s, 1, Nb, 1e-9).kept(0).tolist() == [int(hi[0])]


def test_mass_rule_brute_force_and_margin():
    rng = np.random.default_rng(7)
    Nb = 24
    s = rng.standard_normal((1, 2, Nb, Nb)) * 2
    tau, cap = 0.7, 9
    sel = oracle.select(s, 1, cap, tau)
    flat = s.reshape(-1, Nb)
    for r in range(flat.shape[0]):
        p = np.exp(flat[r] - flat[r].max()); p /= p.sum()
        order = sorted(range(Nb), key=lambda j: (-flat[r, j], j))
        cum = np.cumsum(p[order])
        n = int(np.argmax(cum >= tau)) + 1
        assert sel.counts[r] == min(n, cap)
        assert sel.kept(r).tolist() == sorted(order[:min(n, cap)])
        # the margin: how close the mass comes to tau at any prefix shorter than the cap (up to the crossing)
        cands = [abs(cum[m - 1] - tau) for m in range(1, min(n, cap - 1) + 1)]
        exp_margin = min(cands) if cands else np.inf
        assert sel.mass_margin[r] == pytest.approx(exp_margin, rel=1e-9)


def test_mass_margin_when_the_crossing_lies_beyond_the_cap():
    """tau = 1 is only reached by all blocks together, so the cap decides the count -- but a peaked row gets
    within rounding of 1 after two blocks, which is where an fp32 implementation stops: the row must be
    reported as a near-tie."""
    Nb, cap = 8, 5
    row = np.array([30.0, 29.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0])
    s = np.tile(row, (1, 1, Nb, 1))
    sel = oracle.select(s, 1, cap, 1.0)
    assert (sel.counts == cap).all()                       # the rule itself: mass < 1 until the last block, capped at 5
    p = np.exp(row - row.max()); p /= p.sum()
    assert sel.mass_margin[0] == pytest.approx(1.0 - np.cumsum(p)[cap - 2], rel=1e-6)
    assert sel.mass_margin[0] < 1e-10
    # a flat row is nowhere near tau before the cap
    sel2 = oracle.select(np.zeros((1, 1, Nb, Nb)), 1, cap, 1.0)
    assert (sel2.counts == cap).all() and (sel2.mass_margin > 0.4).all()


def test_forced_window_hand_enumerated():
    # 3 frames x 4 strips; window 3x3 clipped at the borders, no wrap-around
    Nb, bpf = 12, 4
    s = np.zeros((1, 1, Nb, Nb))
    s[0, 0, :, :] = -np.arange(Nb)[None, :]          # scores prefer low indices
    sel = oracle.select(s, 0, 7, win_t=1, win_s=1, blocks_per_frame=bpf)
    corner = sel.kept(0).tolist()      # (t0,s0): forced {0,1,4,5}; then best unforced 2,3,6
    assert corner == [0, 1, 2, 3, 4, 5, 6]
    edge = sel.kept(2).tolist()        # (t0,s2): forced {1,2,3,5,6,7}; then 0
    assert edge == [0, 1, 2, 3, 5, 6, 7]
    interior = sel.kept(5).tolist()    # (t1,s1): forced 0,1,2,4,5,6,8,9,10 = 9 > k=7 -> all 9 kept
    assert interior == [0, 1, 2, 4, 5, 6, 8, 9, 10]
    last = sel.kept(11).tolist()       # (t2,s3): forced {6,7,10,11}; then 0,1,2
    assert last == [0, 1, 2, 6, 7, 10, 11]
    # strips do not wrap: row 4 = (t1,s0) must not force block 3 = (t0,s3)
    r4 = oracle.select(s, 0, 6, win_t=1, win_s=1, blocks_per_frame=bpf).kept(4).tolist()
    assert r4 == [0, 1, 4, 5, 8, 9]
    # invariants: F(I) is a subset of kept(I); count == k whenever |F| <= k
    for I in range(Nb):
        t, st = divmod(I, bpf)
        F = {(t + a) * bpf + (st + b) for a in (-1, 0, 1) for b in (-1, 0, 1)
             if 0 <= t + a < 3 and 0 <= st + b < bpf}
        assert F <= set(sel.kept(I).tolist())
        assert sel.counts[I] == max(7, len(F))
    # window with the mass rule: forced mass counts, count never below |F|
    selm = oracle.select(s, 1, 12, 1e-6, win_t=0, win_s=1, blocks_per_frame=bpf)
    assert selm.kept(6).tolist() == [5, 6, 7]


def test_select_from_qk_end_to_end_integer_inputs():
    """Pool -> score -> top-k on inputs whose scores are exact integers."""
    block = 8
    u = np.array([[1, 0], [0, 1], [1, 1], [2, -1]], float)
    w = np.array([[3, 0], [0, 3], [1, 1], [3, 3]], float)
    q, k = _block_const(u, block), _block_const(w, block)
    sel, s = oracle.select_from_qk(q, k, 32, block, 1.0, 0, 2)
    np.testing.assert_array_equal(s[0, 0], u @ w.T)
    # rows: [3,0,1,3] -> {0,3}; [0,3,1,3] -> {1,3}; [3,3,2,6] -> {0,3} (tie 0 vs 1 -> 0); [6,-3,1,3] -> {0,3}
    assert [sel.kept(r).tolist() for r in range(4)] == [[0, 3], [1, 3], [0, 3], [0, 3]]
