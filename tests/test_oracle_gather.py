"""Pins of the oracle's token gather / scatter against facts that do not go through it."""
import numpy as np

import oracle


def test_gather_matches_the_library_take_and_known_values():
    rng = np.random.default_rng(3)
    x = rng.integers(0, 1 << 16, size=(2, 3, 11, 8)).astype(np.uint16)
    idx = np.stack([rng.permutation(11)[:6], rng.permutation(11)[:6]]).astype(np.int32)
    g = oracle.gather_tokens(x, idx)
    for b in range(2):
        np.testing.assert_array_equal(g[b], np.take(x[b], idx[b], axis=1))
    # a hand-written case: rows are their own index
    y = np.broadcast_to(np.arange(5, dtype=np.float64)[None, None, :, None], (1, 2, 5, 4)).copy()
    np.testing.assert_array_equal(oracle.gather_tokens(y, np.array([[4, 0, 2]], np.int32))[0, 1, :, 0], [4.0, 0.0, 2.0])
    # identity subset = copy
    np.testing.assert_array_equal(oracle.gather_tokens(x, np.tile(np.arange(11, dtype=np.int32), (2, 1))), x)


def test_scatter_inverts_gather_and_leaves_other_rows_alone():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 2, 9, 4))
    idx = np.stack([np.sort(rng.permutation(9)[:5]), np.sort(rng.permutation(9)[:5])]).astype(np.int32)
    back = oracle.scatter_tokens(oracle.gather_tokens(x, idx), idx, np.full_like(x, -7.0))
    for b in range(2):
        kept = np.zeros(9, bool); kept[idx[b]] = True
        np.testing.assert_array_equal(back[b][:, kept], x[b][:, kept])
        assert (back[b][:, ~kept] == -7.0).all()
    # a permutation and its inverse
    perm = rng.permutation(9).astype(np.int32)
    inv = np.argsort(perm).astype(np.int32)
    z = oracle.gather_tokens(oracle.gather_tokens(x[:1], perm[None]), inv[None])
    np.testing.assert_array_equal(z, x[:1])
