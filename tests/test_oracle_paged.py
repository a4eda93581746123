"""Pins of the paged-cache attention oracle (CPU only).

The paged form is a storage layout: the result must not depend on where the pages sit.  It is pinned against
(1) an independent numpy evaluation of the definition on a tiny case, reading the pages through the table itself,
(2) the contiguous oracle on the same keys and values, and (3) invariance under a re-shuffle of the page pool.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2401_15077_b200 import workloads as W


def _f64(x):
    return x.to(torch.float64).numpy()


def _tiny():
    cfg = W.VerifyConfig("paged_tiny", 41, 3, 4, 2, 16, (5, 40), (1, 9), 4, 0, 64, "none")
    return cfg, W.make_attn_inputs(cfg, salt=3)


@pytest.mark.parametrize("page_size", [4, 16, 64])
def test_matches_numpy_definition(page_size):
    cfg, inp = _tiny()
    pk = W.make_paged_cache(inp, page_size, salt=1)
    got = oracle.tree_verify_attn_paged(inp.q, pk.k_pages, pk.v_pages, pk.block_table, inp.seq_lens, inp.tree_parent,
                                        inp.tree_sizes)
    q, kp, vp = _f64(inp.q), _f64(pk.k_pages), _f64(pk.v_pages)
    G = cfg.num_q_heads // cfg.num_kv_heads
    for b in range(cfg.batch):
        L, n = int(inp.seq_lens[b]), int(inp.tree_sizes[b])
        for i in range(cfg.max_tree):
            for h in range(cfg.num_q_heads):
                if i >= n:
                    assert np.all(got[b, i, h] == 0.0)
                    continue
                slots = list(range(L))
                c = i
                while c >= 0:
                    slots.append(L + c)
                    c = int(inp.tree_parent[b, c])
                pages = [int(pk.block_table[b, j // page_size]) for j in slots]
                rows = [j % page_size for j in slots]
                K = kp[pages, h // G, rows]
                V = vp[pages, h // G, rows]
                s = K @ q[b, i, h] / np.sqrt(cfg.head_dim)
                w = np.exp(s - s.max())
                ref = (w / w.sum()) @ V
                np.testing.assert_allclose(got[b, i, h], ref, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("page_size", [8, 128])
def test_equals_contiguous_oracle(page_size):
    cfg, inp = _tiny()
    pk = W.make_paged_cache(inp, page_size, salt=2)
    a = oracle.tree_verify_attn_paged(inp.q, pk.k_pages, pk.v_pages, pk.block_table, inp.seq_lens, inp.tree_parent,
                                      inp.tree_sizes)
    b = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    assert np.array_equal(a, b)


def test_independent_of_page_placement():
    cfg, inp = _tiny()
    outs = []
    for salt in (5, 6):
        pk = W.make_paged_cache(inp, 16, salt=salt, spare_pages=salt)
        outs.append(oracle.tree_verify_attn_paged(inp.q, pk.k_pages, pk.v_pages, pk.block_table, inp.seq_lens,
                                                  inp.tree_parent, inp.tree_sizes))
    assert np.array_equal(outs[0], outs[1])


def test_rejects_a_visible_slot_without_a_page():
    cfg, inp = _tiny()
    pk = W.make_paged_cache(inp, 16, salt=1)
    bad = pk.block_table.clone()
    bad[1, 0] = pk.k_pages.shape[0]
    with pytest.raises(ValueError):
        oracle.tree_verify_attn_paged(inp.q, pk.k_pages, pk.v_pages, bad, inp.seq_lens, inp.tree_parent, inp.tree_sizes)


# ---- commit of the accepted path on a paged cache: expected values come from how the pages were filled

def _paged_commit_case(rng, page_size, T=5, Hkv=2, D=8):
    import itertools
    paths = [list(c) for r in range(T + 1) for c in itertools.combinations(range(T), r)]
    B = len(paths)
    lens = rng.integers(0, 3 * page_size, size=B).astype(np.int32)
    per_seq = int((lens.max() + T + page_size - 1) // page_size) + 1
    need = [int((lens[b] + T + page_size - 1) // page_size) for b in range(B)]
    P = sum(need) + 2
    order = rng.permutation(P)
    table = np.full((B, per_seq), -1, np.int32)
    nxt = 0
    for b in range(B):
        for i in range(need[b]):
            table[b, i] = order[nxt]
            nxt += 1
    k = rng.integers(0, 2 ** 16, size=(P, Hkv, page_size, D), dtype=np.uint16)
    v = rng.integers(0, 2 ** 16, size=(P, Hkv, page_size, D), dtype=np.uint16)
    out = np.full((B, T), -1, np.int32)
    for b, p in enumerate(paths):
        out[b, :len(p)] = p
    return paths, lens, table, k, v, out


def _slot(pages, table, b, j, page_size):
    return pages[table[b, j // page_size], :, j % page_size]


@pytest.mark.parametrize("page_size", [2, 4, 16])
def test_paged_commit_every_increasing_path(page_size):
    rng = np.random.default_rng(10 + page_size)
    T = 5
    paths, lens, table, k, v, padded = _paged_commit_case(rng, page_size, T=T)
    res = oracle.tree_commit_paged(k, v, table, lens, padded, T)
    touched = np.zeros(k.shape[:1] + k.shape[2:3], bool)       # (page, row) pairs that may change
    for b, p in enumerate(paths):
        L, a = int(lens[b]), len(p)
        assert res["valid"][b] == 1 and res["new_seq_lens"][b] == L + a
        for new, old in ((res["k_pages"], k), (res["v_pages"], v)):
            for j, m in enumerate(p):
                assert np.array_equal(_slot(new, table, b, L + j, page_size), _slot(old, table, b, L + m, page_size)), (p, j)
        for j in range(a):
            touched[table[b, (L + j) // page_size], (L + j) % page_size] = True
    for new, old in ((res["k_pages"], k), (res["v_pages"], v)):
        same = np.all(new == old, axis=(1, 3))
        assert same[~touched].all(), "rows outside the committed slots must not change"


def test_paged_commit_equals_contiguous_commit():
    """Gathering the pages into a contiguous cache commutes with the commit."""
    rng = np.random.default_rng(3)
    T, ps = 5, 4
    paths, lens, table, k, v, padded = _paged_commit_case(rng, ps, T=T)
    B, per_seq = table.shape
    cap = per_seq * ps

    def gather(pages):
        out = np.zeros((B, pages.shape[1], cap, pages.shape[3]), np.uint16)
        for b in range(B):
            for i in range(per_seq):
                if table[b, i] >= 0:
                    out[b, :, i * ps:(i + 1) * ps] = pages[table[b, i]]
        return out

    paged = oracle.tree_commit_paged(k, v, table, lens, padded, T)
    flat = oracle.tree_commit(gather(k), gather(v), lens, padded, T)
    assert np.array_equal(gather(paged["k_pages"]), flat["k_cache"])
    assert np.array_equal(gather(paged["v_pages"]), flat["v_cache"])
    assert np.array_equal(paged["new_seq_lens"], flat["new_seq_lens"])


def test_paged_commit_invalid_rows_are_left_alone():
    rng = np.random.default_rng(4)
    T, ps = 5, 4
    paths, lens, table, k, v, padded = _paged_commit_case(rng, ps, T=T)
    bad_path, bad_page = 7, 20
    padded[bad_path, :2] = (3, 1)                                   # not increasing
    L = int(lens[bad_page])
    padded[bad_page, :] = -1
    padded[bad_page, :2] = (0, 4)
    table[bad_page, (L + 4) // ps] = k.shape[0] + 3                  # the source slot's page does not exist
    res = oracle.tree_commit_paged(k, v, table, lens, padded, T)
    for b in (bad_path, bad_page):
        assert res["valid"][b] == 0 and res["new_seq_lens"][b] == lens[b]
    # the invalid sequences' pages are unchanged
    for b in (bad_path, bad_page):
        for i in range(table.shape[1]):
            if 0 <= table[b, i] < k.shape[0]:
                assert np.array_equal(res["k_pages"][table[b, i]], k[table[b, i]])
