"""Pins for the oracle's tree mask and tree attention (CPU only).

The oracle is checked against things other than itself: library attention routines on the special
cases that reduce to them, closed forms, brute force over every small tree, and invariants that
follow from the definition of tree attention (Sec. 3.3, App. A.1: a draft token attends to the
committed context and to the tokens on its own root path).
"""
import itertools

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_2401_15077_b200 import workloads as W


def _rand_case(B, T, Hq, Hkv, D, lens, parents, seed=0, sizes=None):
    g = torch.Generator().manual_seed(seed)
    cap = max(int(l) for l in lens) + T + 3
    q = torch.randn((B, T, Hq, D), generator=g).to(torch.bfloat16)
    k = torch.randn((B, Hkv, cap, D), generator=g).to(torch.bfloat16)
    v = torch.randn((B, Hkv, cap, D), generator=g).to(torch.bfloat16)
    sl = torch.tensor(lens, dtype=torch.int32)
    par = torch.tensor(parents, dtype=torch.int32)
    ts = None if sizes is None else torch.tensor(sizes, dtype=torch.int32)
    return q, k, v, sl, par, ts


def _closure_mask(parent):
    """Ancestor-or-self matrix by repeated squaring of (I + adjacency): independent of the oracle's walk."""
    T = len(parent)
    A = np.eye(T, dtype=np.int64)
    for i, p in enumerate(parent):
        if p >= 0:
            A[i, p] = 1
    R = A.copy()
    for _ in range(max(1, T.bit_length())):
        R = ((R @ R) > 0).astype(np.int64)
    return R.astype(bool)


def _sdpa_reference(q, k, v, sl, par, scale=None):
    """torch scaled_dot_product_attention in float64 with an explicit boolean mask (one sequence)."""
    B, T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    outs = []
    for b in range(B):
        L = int(sl[b])
        keys = k[b, :, :L + T].double().repeat_interleave(G, dim=0)
        vals = v[b, :, :L + T].double().repeat_interleave(G, dim=0)
        qq = q[b].double().permute(1, 0, 2)  # [Hq, T, D]
        m = torch.zeros((T, L + T), dtype=torch.bool)
        m[:, :L] = True
        m[:, L:] = torch.from_numpy(_closure_mask([int(x) for x in par[b]]))
        outs.append(F.scaled_dot_product_attention(qq, keys, vals, attn_mask=m, scale=scale).permute(1, 0, 2))
    return torch.stack(outs).numpy()


# ------------------------------------------------------------------------------------------ mask

@pytest.mark.parametrize("T", [1, 2, 3, 4, 5, 6])
def test_ancestors_brute_force_all_trees(oracle, T):
    trees = list(itertools.product(*[range(-1, i) for i in range(T)]))
    assert len(trees) == [1, 2, 6, 24, 120, 720][T - 1]
    par = np.array(trees, dtype=np.int32)
    anc, depth = oracle.tree_ancestors(par)
    for t, a, d in zip(trees, anc, depth):
        ref = _closure_mask(list(t))
        for i in range(T):
            bits = [(int(a[i]) >> j) & 1 for j in range(T)]
            assert bits == [int(x) for x in ref[i]]
            assert bin(int(a[i])).count("1") == d[i]
            assert int(a[i]) >> (i + 1) == 0 and (int(a[i]) >> i) & 1
            if t[i] >= 0:
                assert int(a[i]) & int(a[t[i]]) == int(a[t[i]])
                assert d[i] == d[t[i]] + 1
            else:
                assert d[i] == 1 and int(a[i]) == 1 << i


def test_ancestors_full_width_chain_and_sizes(oracle):
    par = np.arange(-1, 63, dtype=np.int32)[None, :]
    anc, depth = oracle.tree_ancestors(par)
    assert [int(x) for x in anc[0]] == [(1 << (i + 1)) - 1 for i in range(64)]
    assert list(depth[0]) == list(range(1, 65))
    par2 = np.array([[-1, 0, 0, 99, 99]], dtype=np.int32)
    anc2, depth2 = oracle.tree_ancestors(par2, np.array([3], np.int32))
    assert [int(x) for x in anc2[0]] == [1, 3, 5, 0, 0] and list(depth2[0]) == [1, 2, 2, 0, 0]


def test_invalid_trees_rejected(oracle):
    with pytest.raises(ValueError):
        oracle.tree_ancestors(np.array([[-1, 1]], np.int32))
    with pytest.raises(ValueError):
        oracle.tree_ancestors(np.array([[-2]], np.int32))


# ------------------------------------------------------------------------------------- attention

def test_chain_tree_is_causal_attention(oracle):
    """A chain draft (no tree attention, App. A.1) must equal causal attention of the last T queries."""
    B, T, H, D, L = 2, 7, 3, 16, 11
    q, k, v, sl, par, _ = _rand_case(B, T, H, H, D, [L, L], [list(range(-1, T - 1))] * B, seed=1)
    out = oracle.tree_verify_attn(q, k, v, sl, par)
    for b in range(B):
        keys = k[b, :, :L + T].double()
        vals = v[b, :, :L + T].double()
        # pad queries in front so that is_causal's top-left alignment gives the last T rows
        qfull = torch.zeros((H, L + T, D), dtype=torch.float64)
        qfull[:, L:] = q[b].double().permute(1, 0, 2)
        ref = F.scaled_dot_product_attention(qfull, keys, vals, is_causal=True)[:, L:].permute(1, 0, 2)
        np.testing.assert_allclose(out[b], ref.numpy(), rtol=1e-12, atol=1e-13)


def test_single_node_is_plain_decode(oracle):
    B, H, D, L = 1, 4, 32, 37
    q, k, v, sl, par, _ = _rand_case(B, 1, H, H, D, [L], [[-1]], seed=2)
    out = oracle.tree_verify_attn(q, k, v, sl, par)
    ref = F.scaled_dot_product_attention(q[0].double().permute(1, 0, 2), k[0, :, :L + 1].double(),
                                         v[0, :, :L + 1].double()).permute(1, 0, 2)
    np.testing.assert_allclose(out[0], ref.numpy(), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_general_tree_matches_masked_library_attention(oracle, seed):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=3, prefix=(0, 40), tree=(1, 12), num_q_heads=4, num_kv_heads=2,
                   head_dim=16)
    inp = W.make_attn_inputs(cfg, salt=seed, poison=False)
    out = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    for b in range(cfg.batch):
        n = int(inp.tree_sizes[b])
        ref = _sdpa_reference(inp.q[b:b + 1, :n], inp.k_cache[b:b + 1, :, :int(inp.seq_lens[b]) + n],
                              inp.v_cache[b:b + 1, :, :int(inp.seq_lens[b]) + n], inp.seq_lens[b:b + 1],
                              inp.tree_parent[b:b + 1, :n])
        np.testing.assert_allclose(out[b, :n], ref[0], rtol=1e-11, atol=1e-12)
        assert np.all(out[b, n:] == 0.0)


def test_scale_override(oracle):
    q, k, v, sl, par, _ = _rand_case(1, 4, 2, 2, 8, [5], [[-1, 0, 0, 2]], seed=3)
    out = oracle.tree_verify_attn(q, k, v, sl, par, sm_scale=0.37)
    ref = _sdpa_reference(q, k, v, sl, par, scale=0.37)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)
    default = oracle.tree_verify_attn(q, k, v, sl, par)
    np.testing.assert_allclose(default, _sdpa_reference(q, k, v, sl, par, scale=8 ** -0.5), rtol=1e-12, atol=1e-13)


def test_closed_forms(oracle):
    parents = [[-1, 0, 0, 1, -1, 4]]
    q, k, v, sl, par, _ = _rand_case(1, 6, 2, 1, 8, [9], parents, seed=4)
    # every value row equal to c  =>  output equals c
    c = torch.arange(8, dtype=torch.float32).to(torch.bfloat16)
    out = oracle.tree_verify_attn(q, k, c.expand_as(v).contiguous(), sl, par)
    np.testing.assert_allclose(out, np.broadcast_to(c.double().numpy(), out.shape), rtol=1e-13)
    # all keys zero  =>  uniform weights: mean of the visible value rows (prefix + depth of them)
    out = oracle.tree_verify_attn(q, torch.zeros_like(k), v, sl, par)
    L = 9
    paths = {0: [0], 1: [0, 1], 2: [0, 2], 3: [0, 1, 3], 4: [4], 5: [4, 5]}
    for i, path in paths.items():
        rows = list(range(L)) + [L + m for m in path]
        ref = v[0, 0, rows].double().mean(dim=0).numpy()
        for h in range(2):
            np.testing.assert_allclose(out[0, i, h], ref, rtol=1e-13, atol=1e-14)


def test_star_tree_is_independent_decodes(oracle):
    T, H, D, L = 5, 2, 16, 13
    q, k, v, sl, par, _ = _rand_case(1, T, H, H, D, [L], [[-1] * T], seed=5)
    out = oracle.tree_verify_attn(q, k, v, sl, par)
    for i in range(T):
        rows = list(range(L)) + [L + i]
        ref = F.scaled_dot_product_attention(q[0, i].double()[:, None, :], k[0][:, rows].double(),
                                             v[0][:, rows].double())[:, 0]
        np.testing.assert_allclose(out[0, i], ref.numpy(), rtol=1e-12, atol=1e-13)


def test_non_ancestors_and_padding_do_not_matter(oracle):
    parents = [[-1, 0, 0, 1, 2, -1]]
    q, k, v, sl, par, _ = _rand_case(1, 6, 2, 2, 8, [4], parents, seed=6)
    base = oracle.tree_verify_attn(q, k, v, sl, par)
    anc = {0: {0}, 1: {0, 1}, 2: {0, 2}, 3: {0, 1, 3}, 4: {0, 2, 4}, 5: {5}}
    for m in range(6):
        k2, v2, q2 = k.clone(), v.clone(), q.clone()
        k2[0, :, 4 + m] += 3.0
        v2[0, :, 4 + m] -= 2.0
        q2[0, m] *= -1.5
        out_kv = oracle.tree_verify_attn(q, k2, v2, sl, par)
        out_q = oracle.tree_verify_attn(q2, k, v, sl, par)
        for i in range(6):
            assert (np.array_equal(out_kv[0, i], base[0, i])) == (m not in anc[i])
            assert (np.array_equal(out_q[0, i], base[0, i])) == (m != i)
    # slots past prefix + tree are never read: NaN there changes nothing
    k3, v3 = k.clone(), v.clone()
    k3[0, :, 10:] = float("nan")
    v3[0, :, 10:] = float("nan")
    assert np.array_equal(oracle.tree_verify_attn(q, k3, v3, sl, par), base)


def test_topological_relabelling_permutes_rows(oracle):
    parents = [-1, 0, 0, 1, 2, -1]
    perm = [0, 2, 1, 5, 4, 3]  # new index of old node; keeps parents before children
    q, k, v, sl, par, _ = _rand_case(1, 6, 1, 1, 8, [3], [parents], seed=7)
    base = oracle.tree_verify_attn(q, k, v, sl, par)
    q2, k2, v2 = q.clone(), k.clone(), v.clone()
    par2 = [0] * 6
    for old, new in enumerate(perm):
        q2[0, new] = q[0, old]
        k2[0, :, 3 + new] = k[0, :, 3 + old]
        v2[0, :, 3 + new] = v[0, :, 3 + old]
        par2[new] = -1 if parents[old] < 0 else perm[parents[old]]
    assert all(p < i for i, p in enumerate(par2))
    out = oracle.tree_verify_attn(q2, k2, v2, sl, torch.tensor([par2], dtype=torch.int32))
    for old, new in enumerate(perm):
        np.testing.assert_allclose(out[0, new], base[0, old], rtol=1e-12, atol=1e-14)


def test_gqa_equals_mha_with_repeated_kv_heads(oracle):
    q, k, v, sl, par, _ = _rand_case(2, 5, 6, 2, 8, [7, 2], [[-1, 0, 1, 1, 0]] * 2, seed=8)
    gqa = oracle.tree_verify_attn(q, k, v, sl, par)
    mha = oracle.tree_verify_attn(q, k.repeat_interleave(3, dim=1), v.repeat_interleave(3, dim=1), sl, par)
    assert np.array_equal(gqa, mha)


def test_empty_prefix_and_empty_tree(oracle):
    q, k, v, sl, par, ts = _rand_case(2, 3, 2, 2, 8, [0, 5], [[-1, 0, -1], [7, 7, 7]], seed=9, sizes=[3, 0])
    out = oracle.tree_verify_attn(q, k, v, sl, par, ts)
    # L = 0, top-level node: softmax over its own key only => its own value row
    np.testing.assert_allclose(out[0, 0], v[0, :, 0].double().numpy(), rtol=1e-13)
    np.testing.assert_allclose(out[0, 2], v[0, :, 2].double().numpy(), rtol=1e-13)
    assert np.all(out[1] == 0.0)
