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
