"""Pins of the oracle's commit of the accepted path (Sec. 3.3: accepted tokens and their features are kept for the next
drafting phase).  The expected values come from how the inputs were built (which tree node's rows were put where), never
from re-running the oracle's own assignment."""
import itertools

import numpy as np
import pytest

from paper_2401_15077_b200 import workloads as W


def _build(rng, B, Hkv, D, T, lens, cap, F=0):
    """A cache whose tree slots hold known per-node rows: returns (k, v, node_k, node_v, feats)."""
    k = rng.integers(0, 2 ** 16, size=(B, Hkv, cap, D), dtype=np.uint16)
    v = rng.integers(0, 2 ** 16, size=(B, Hkv, cap, D), dtype=np.uint16)
    node_k = rng.integers(0, 2 ** 16, size=(B, Hkv, T, D), dtype=np.uint16)
    node_v = rng.integers(0, 2 ** 16, size=(B, Hkv, T, D), dtype=np.uint16)
    for b in range(B):
        k[b, :, lens[b]:lens[b] + T] = node_k[b]
        v[b, :, lens[b]:lens[b] + T] = node_v[b]
    feats = rng.integers(0, 2 ** 16, size=(B, T, F), dtype=np.uint16) if F else None
    return k, v, node_k, node_v, feats


def _pad(paths, cap):
    out = np.full((len(paths), cap), -1, np.int32)
    for b, p in enumerate(paths):
        out[b, :len(p)] = p
    return out


def test_every_increasing_path_of_a_small_tree(oracle):
    """All 32 increasing node subsets of a 5-node tree, as 32 sequences of one call: afterwards the prefix is the old prefix
    followed by the accepted nodes' rows in path order (known from the construction), everything else is untouched."""
    T, Hkv, D, F = 5, 2, 8, 6
    paths = [list(c) for r in range(T + 1) for c in itertools.combinations(range(T), r)]
    B = len(paths)
    rng = np.random.default_rng(1)
    lens = rng.integers(0, 7, size=B).astype(np.int32)
    cap = int(lens.max()) + T + 2
    k, v, node_k, node_v, feats = _build(rng, B, Hkv, D, T, lens, cap, F)
    res = oracle.tree_commit(k, v, lens, _pad(paths, T), T, features=feats)
    for b, p in enumerate(paths):
        L, a = int(lens[b]), len(p)
        assert res["valid"][b] == 1 and res["new_seq_lens"][b] == L + a
        for new, old, node in ((res["k_cache"], k, node_k), (res["v_cache"], v, node_v)):
            assert np.array_equal(new[b, :, :L], old[b, :, :L])
            for j, m in enumerate(p):
                assert np.array_equal(new[b, :, L + j], node[b, :, m]), (p, j)
            assert np.array_equal(new[b, :, L + a:], old[b, :, L + a:])
        for j, m in enumerate(p):
            assert np.array_equal(res["features_out"][b, j], feats[b, m])
        assert not res["features_out"][b, a:].any()


def test_chain_path_changes_nothing(oracle):
    """Accepting nodes 0, 1, 2, ... in place is the identity on the cache (the rows already sit where they belong)."""
    rng = np.random.default_rng(2)
    B, Hkv, D, T = 3, 2, 16, 9
    lens = np.array([0, 5, 11], np.int32)
    k, v, *_ = _build(rng, B, Hkv, D, T, lens, 24)
    res = oracle.tree_commit(k, v, lens, _pad([list(range(9)), list(range(4)), []], 9), T)
    assert np.array_equal(res["k_cache"], k) and np.array_equal(res["v_cache"], v)
    assert res["new_seq_lens"].tolist() == [9, 9, 11]


def test_sources_that_are_also_destinations(oracle):
    """path = (1, 2, 3): slot L+1 is read for position 0 and written for position 1.  A copy in descending order would
    hand node 3's rows to every position; the assignment is simultaneous."""
    rng = np.random.default_rng(3)
    lens = np.array([4], np.int32)
    k, v, node_k, node_v, _ = _build(rng, 1, 1, 8, 6, lens, 12)
    res = oracle.tree_commit(k, v, lens, _pad([[1, 2, 3]], 6), 6)
    for j, m in enumerate((1, 2, 3)):
        assert np.array_equal(res["k_cache"][0, 0, 4 + j], node_k[0, 0, m])
        assert np.array_equal(res["v_cache"][0, 0, 4 + j], node_v[0, 0, m])


def test_entries_after_the_first_minus_one_are_ignored_and_path_cap_may_exceed_the_tree(oracle):
    rng = np.random.default_rng(4)
    lens = np.array([2], np.int32)
    k, v, node_k, *_ = _build(rng, 1, 1, 8, 4, lens, 8)
    path = np.array([[2, -1, 3, 1, -1, -1, -1]], np.int32)
    res = oracle.tree_commit(k, v, lens, path, 4)
    assert res["new_seq_lens"][0] == 3 and np.array_equal(res["k_cache"][0, 0, 2], node_k[0, 0, 2])
    assert np.array_equal(res["k_cache"][0, 0, 3:], k[0, 0, 3:])


@pytest.mark.parametrize("bad", [[3, 2], [1, 1], [0, 7], [5], [-2]])
def test_invalid_paths_leave_the_sequence_alone(oracle, bad):
    """Not increasing, outside the tree, below -1, or pointing past the cache: nothing moves, the length stays, valid = 0;
    the neighbouring sequence is still committed."""
    rng = np.random.default_rng(5)
    T = 7 if bad != [5] else 8
    lens = np.array([3, 3], np.int32)
    cap = 8 if bad == [5] else 12            # [5]: slot 3 + 5 = 8 does not exist
    k, v, node_k, _, feats = _build(rng, 2, 2, 8, min(T, cap - 3), lens, cap, 4)
    feats = rng.integers(0, 2 ** 16, size=(2, T, 4), dtype=np.uint16)
    res = oracle.tree_commit(k, v, lens, _pad([bad, [1]], 3), T, features=feats)
    assert res["valid"].tolist() == [0, 1] and res["new_seq_lens"].tolist() == [3, 4]
    assert np.array_equal(res["k_cache"][0], k[0]) and np.array_equal(res["v_cache"][0], v[0])
    assert not res["features_out"][0].any()
    assert np.array_equal(res["k_cache"][1, :, 3], node_k[1, :, 1])


def test_generated_paths_are_chains_of_their_trees(oracle):
    """The input generator's paths are root-to-node chains (each entry's parent is the entry before it), so they are what
    an acceptance walk can produce; the oracle accepts every one of them."""
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=40, prefix=(0, 50))
    sizes, parent = W.make_trees(cfg, salt=3)
    paths = W.make_accepted_paths(sizes, parent, cfg.max_tree, cfg.index, salt=3).numpy()
    lens = np.zeros(40, np.int32)
    assert (paths[:, 0] >= 0).sum() > 10
    for b in range(40):
        prev = -1
        for m in paths[b]:
            if m < 0:
                break
            assert int(parent[b, m]) == prev and m < int(sizes[b])
            prev = int(m)
    rng = np.random.default_rng(6)
    k, v, *_ = _build(rng, 40, 1, 8, cfg.max_tree, lens, cfg.max_tree)
    assert oracle.tree_commit(k, v, lens, paths, cfg.max_tree)["valid"].all()
