"""Pins of the oracle's child selection for draft-tree nodes (App. A.1: top-k children in the greedy setting, k sampled
children otherwise)."""
import numpy as np
from scipy import stats


def _rows(seed, B=6, R=5, V=301):
    rng = np.random.default_rng(seed)
    return rng.dirichlet(np.full(V, 0.3), size=(B, R)).astype(np.float32)


def test_top_k_equals_a_library_sort(oracle):
    """numpy's stable argsort of -p gives descending probability with the lower id first among equals."""
    p = _rows(1)
    p[0, 0, 10:20] = p[0, 0, 5]            # ties inside the top
    p[1, 2, :] = 1.0 / p.shape[2]          # a constant row: ids 0..k-1
    B, R, V = p.shape
    K = 9
    nc = np.random.default_rng(2).integers(0, K + 1, size=(B, R)).astype(np.int32)
    nc[0, 0], nc[1, 2] = K, K
    res = oracle.tree_expand(p, nc, K, greedy=np.ones(B, np.uint8))
    for b in range(B):
        for r in range(R):
            k = nc[b, r]
            want = np.argsort(-p[b, r], kind="stable")[:k]
            assert res["tokens"][b, r, :k].tolist() == want.tolist()
            assert (res["tokens"][b, r, k:] == -1).all() and (res["token_probs"][b, r, k:] == 0).all()
            assert np.array_equal(res["token_probs"][b, r, :k], p[b, r, want])
    assert res["tokens"][1, 2].tolist() == list(range(K))


def test_draws_are_the_inverse_cdf_of_each_uniform(oracle):
    """A row with masses (1, 0, 2, 0, 1) / 4: cells [0, .25), [.25, .75), [.75, 1); zero-mass tokens are never drawn; every draw
    depends on its own uniform only (with replacement)."""
    p = np.zeros((1, 1, 5), np.float32)
    p[0, 0] = [0.25, 0, 0.5, 0, 0.25]
    un = np.array([[[0.0, 0.2499, 0.25, 0.6, 0.7499, 0.75, 0.999, 0.6]]], np.float32)
    res = oracle.tree_expand(p, np.array([[8]], np.int32), 8, uniforms=un)
    assert res["tokens"][0, 0].tolist() == [0, 0, 2, 2, 2, 4, 4, 2]
    assert np.allclose(res["token_probs"][0, 0], [0.25, 0.25, 0.5, 0.5, 0.5, 0.25, 0.25, 0.5])
    assert abs(res["min_margin"][0, 0] - 0.0) < 1e-6          # u = 0.25 sits on an edge (the cell's own lower edge)


def test_unnormalised_rows_are_used_as_given(oracle):
    p = _rows(3, B=2, R=3)
    un = np.random.default_rng(4).random((2, 3, 6), dtype=np.float32)
    nc = np.full((2, 3), 6, np.int32)
    a = oracle.tree_expand(p, nc, 6, uniforms=un)
    b = oracle.tree_expand(p * np.float32(4.0), nc, 6, uniforms=un)      # exact scaling by a power of two
    assert np.array_equal(a["tokens"], b["tokens"])


def test_draws_follow_the_row_distribution(oracle):
    """Chi-square over 2e5 draws of a 12-token row (16 draws per node, 12500 nodes with the same row)."""
    V, n, K = 12, 12500, 16
    rng = np.random.default_rng(5)
    row = rng.dirichlet(np.ones(V)).astype(np.float32)
    p = np.broadcast_to(row, (n, 1, V)).copy()
    un = rng.random((n, 1, K), dtype=np.float32)
    res = oracle.tree_expand(p, np.full((n, 1), K, np.int32), K, uniforms=un)
    counts = np.bincount(res["tokens"].ravel(), minlength=V)
    pr = row.astype(np.float64) / row.astype(np.float64).sum()
    assert stats.chisquare(counts, pr * n * K).pvalue > 1e-3


def test_mixed_batch_and_zero_children(oracle):
    p = _rows(6, B=4, R=3)
    gr = np.array([1, 0, 1, 0], np.uint8)
    nc = np.array([[0, 2, 4], [3, 0, 1], [1, 1, 0], [0, 0, 0]], np.int32)
    un = np.random.default_rng(7).random((4, 3, 4), dtype=np.float32)
    res = oracle.tree_expand(p, nc, 4, uniforms=un, greedy=gr)
    assert ((res["tokens"] >= 0).sum(-1) == nc).all()
    assert res["tokens"][0, 2, 0] == p[0, 2].argmax() and np.isinf(res["min_margin"][0, 2])
    cdf = np.cumsum(p[1, 0].astype(np.float64))
    for j in range(3):
        assert res["tokens"][1, 0, j] == np.searchsorted(cdf, np.float64(un[1, 0, j]) * cdf[-1], side="right")
