"""Pins of the oracle's acceptance walk on logits (rows = softmax(logits / temperature), fp64)."""
import numpy as np
import pytest
from scipy import special, stats

from paper_2401_15077_b200 import workloads as W


def _inputs(seed, B=40, T=12, V=257, grid=True):
    rng = np.random.default_rng(seed)
    cfg = W.scaled(W.CONFIGS["tiny"], batch=B, tree=(0, T), vocab=V)
    sizes, parent = W.make_trees(cfg, salt=seed)
    T_max = cfg.max_tree
    # logits on a grid of 1/32 so that adding a power of two or doubling them is exact in fp32
    zt = rng.integers(-160, 161, size=(B, T_max + 1, V)).astype(np.float32) / 32
    zd = (zt[:, :T_max] * 0.75 + rng.integers(-80, 81, size=(B, T_max, V)).astype(np.float32) / 32).astype(np.float32)
    zd = np.round(zd * 32) / 32
    tok = rng.integers(0, V, size=(B, T_max)).astype(np.int32)
    un = rng.random((B, T_max + 1), dtype=np.float32)
    return dict(zt=zt, zd=zd.astype(np.float32), tok=tok, par=parent.numpy(), un=un, sizes=sizes.numpy(), T=T_max, V=V, B=B)


def _walk(oracle, d, zt, zd, temperature, **kw):
    return oracle.tree_accept_logits(zt, zd, d["tok"], d["par"], d["un"], temperature, tree_sizes=d["sizes"], **kw)


def _same(a, b):
    return all(np.array_equal(a[k], b[k]) for k in ("accepted_path", "bonus_token", "accept_len"))


def test_adding_a_constant_to_a_row_changes_nothing(oracle):
    d = _inputs(1)
    base = _walk(oracle, d, d["zt"], d["zd"], 1.0)
    rng = np.random.default_rng(2)
    ct = rng.choice([-16.0, 8.0, 32.0], size=(d["B"], d["T"] + 1, 1)).astype(np.float32)
    cd = rng.choice([-8.0, 4.0, 64.0], size=(d["B"], d["T"], 1)).astype(np.float32)
    shifted = _walk(oracle, d, d["zt"] + ct, d["zd"] + cd, 1.0)
    assert _same(base, shifted) and np.array_equal(base["min_margin"], shifted["min_margin"])
    assert base["accept_len"].max() >= 2 and (base["accept_len"] == 0).any()


@pytest.mark.parametrize("temperature", [0.5, 1.0, 2.0])
def test_scaling_logits_and_temperature_together_changes_nothing(oracle, temperature):
    d = _inputs(3)
    a = _walk(oracle, d, d["zt"], d["zd"], temperature)
    b = _walk(oracle, d, d["zt"] * 4, d["zd"] * 4, temperature * 4)
    assert _same(a, b) and np.array_equal(a["min_margin"], b["min_margin"])


@pytest.mark.parametrize("temperature", [0.7, 1.0, 1.6])
def test_equals_the_probability_walk_on_library_softmax_rows(oracle, temperature):
    """scipy's softmax of logits / T, rounded to fp32, through the (separately pinned) probability walk: same tokens
    unless a decision sits within the fp32 rounding of the rows."""
    d = _inputs(4, B=120)
    got = _walk(oracle, d, d["zt"], d["zd"], temperature)
    pt = special.softmax(d["zt"].astype(np.float64) / temperature, axis=-1).astype(np.float32)
    pd = special.softmax(d["zd"].astype(np.float64) / temperature, axis=-1).astype(np.float32)
    ref = oracle.tree_accept(pt, pd, d["tok"], d["par"], d["un"], tree_sizes=d["sizes"])
    differ = [b for b in range(d["B"]) if not (np.array_equal(got["accepted_path"][b], ref["accepted_path"][b])
                                               and got["bonus_token"][b] == ref["bonus_token"][b])]
    assert all(min(got["min_margin"][b], ref["min_margin"][b]) < 1e-6 for b in differ), differ
    assert len(differ) <= 2
    # the temperature matters: another one gives other tokens
    other = _walk(oracle, d, d["zt"], d["zd"], temperature * 3)
    assert not _same(got, other)


def test_uniform_rows_accept_the_first_child_down_to_a_leaf(oracle):
    """All logits equal: p = p^ = 1/V, so r * p^(t) < p(t) for every r < 1: the walk takes the first child at every node;
    the extra token is the inverse CDF of the uniform distribution, floor(u * V)."""
    d = _inputs(5, B=30, V=64)
    zt = np.full_like(d["zt"], 3.25)
    zd = np.full_like(d["zd"], -1.5)
    res = _walk(oracle, d, zt, zd, 1.3)
    for b in range(d["B"]):
        cur, want = -1, []
        while True:
            kids = [i for i in range(d["sizes"][b]) if d["par"][b, i] == cur]
            if not kids:
                break
            cur = kids[0]
            want.append(cur)
        assert res["accepted_path"][b, :len(want)].tolist() == want and res["accept_len"][b] == len(want)
        u = float(d["un"][b, d["T"]])
        assert abs(int(res["bonus_token"][b]) - int(np.floor(u * 64))) <= (1 if abs(u * 64 - round(u * 64)) < 1e-9 else 0)


def test_first_emitted_token_follows_the_target_softmax_at_the_temperature(oracle):
    """Chi-square on 16 tokens: 3 children of the context whose tokens are re-drawn from softmax(draft / T) in every
    trial; the first emitted token must be distributed as softmax(target / T) (Sec. 3.3: the target distribution is
    preserved), and NOT as the softmax at temperature 1."""
    V, n, T, temperature = 16, 100_000, 3, 0.6
    rng = np.random.default_rng(7)
    zt_root = rng.normal(0, 1.4, size=V).astype(np.float32)
    zd_root = (0.8 * zt_root + rng.normal(0, 0.8, size=V)).astype(np.float32)
    q = special.softmax(zd_root.astype(np.float64) / temperature)
    tokens = np.searchsorted(np.cumsum(q), rng.random((n, T)), side="right").clip(0, V - 1).astype(np.int32)
    zt = np.broadcast_to(zt_root, (n, T + 1, V)).copy()
    zd = np.broadcast_to(zd_root, (n, T, V)).copy()
    parent = np.full((n, T), -1, np.int32)
    un = rng.random((n, T + 1), dtype=np.float32)
    res = oracle.tree_accept_logits(zt, zd, tokens, parent, un, temperature)
    first = np.where(res["accept_len"] > 0, tokens[np.arange(n), np.maximum(res["accepted_path"][:, 0], 0)], res["bonus_token"])
    counts = np.bincount(first, minlength=V)
    p_T = special.softmax(zt_root.astype(np.float64) / temperature)
    assert stats.chisquare(counts, p_T * n).pvalue > 1e-3
    assert stats.chisquare(counts, special.softmax(zt_root.astype(np.float64)) * n).pvalue < 1e-6


def test_greedy_sequences_ignore_the_temperature(oracle):
    d = _inputs(8)
    gr = np.ones(d["B"], np.uint8)
    a = oracle.tree_accept_logits(d["zt"], None, d["tok"], d["par"], None, 0.3, tree_sizes=d["sizes"], greedy=gr)
    b = oracle.tree_accept_logits(d["zt"], None, d["tok"], d["par"], None, 5.0, tree_sizes=d["sizes"], greedy=gr)
    assert _same(a, b)
    am = d["zt"][:, 0].argmax(-1)
    first_kids = [[i for i in range(d["sizes"][s]) if d["par"][s, i] == -1 and d["tok"][s, i] == am[s]] for s in range(d["B"])]
    for s in range(d["B"]):
        if not first_kids[s]:
            assert a["accept_len"][s] == 0 and a["bonus_token"][s] == am[s]
