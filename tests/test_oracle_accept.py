"""Pins for the oracle's acceptance walk (CPU only).

Algorithm 1 (multi-round speculative sampling, App. A.2) is restated here with exact rational
arithmetic as a map "candidates -> outcome distribution"; that restatement is checked against the
theorem the paper relies on (the output is distributed as the target), and the C oracle is then
checked against it region by region, by Monte Carlo, against the closed forms of chain speculative
sampling (Preliminaries), by brute force on small trees, and by a chi-square test on a 16-token
vocabulary.
"""
import itertools
import math
from fractions import Fraction as Fr

import numpy as np
import pytest
from scipy import stats

from paper_2401_15077_b200 import workloads as W


# ----------------------------------------------------------------- exact model of Algorithm 1

def alg1_exact(p, cands):
    """Outcome distribution of Algorithm 1 for a fixed candidate list [(token, p_hat), ...].

    Returns (accept_prob_per_candidate, reach_prob_of_final_draw, final_distribution, thresholds).
    """
    p = list(p)
    reach = Fr(1)
    acc, thresholds = [], []
    for t, q in cands:
        if q[t] > 0:
            a = min(Fr(1), p[t] / q[t])
        else:
            a = Fr(1) if p[t] > 0 else Fr(0)
        thresholds.append(a)
        acc.append(reach * a)
        reach *= 1 - a
        res = [max(Fr(0), pv - qv) for pv, qv in zip(p, q)]
        Z = sum(res)
        if Z > 0:
            p = [r / Z for r in res]
    return acc, reach, p, thresholds


def alg1_token_distribution(p, cands):
    acc, reach, pf, _ = alg1_exact(p, cands)
    out = [Fr(0)] * len(p)
    for (t, _), a in zip(cands, acc):
        out[t] += a
    for v, pv in enumerate(pf):
        out[v] += reach * pv
    return out


P4 = [Fr(1, 2), Fr(1, 4), Fr(1, 8), Fr(1, 8)]
Q4 = [Fr(1, 8), Fr(3, 8), Fr(1, 4), Fr(1, 4)]
# a pair whose residual max(0, p - q) = (1/4, 0, 1/8, 0) keeps two tokens alive after a rejection
P4B = [Fr(3, 8), Fr(1, 8), Fr(3, 8), Fr(1, 8)]


@pytest.mark.parametrize("k", [0, 1, 2, 3])
def test_reading_of_algorithm1_preserves_target_iid(k):
    """Candidates drawn i.i.d. from p_hat: sum over draws of P(draw) * outcome == p exactly."""
    total = [Fr(0)] * 4
    for toks in itertools.product(range(4), repeat=k):
        w = Fr(1)
        for t in toks:
            w *= Q4[t]
        d = alg1_token_distribution(P4B, [(t, Q4) for t in toks])
        total = [a + w * b for a, b in zip(total, d)]
    assert total == P4B


def _without_replacement_rows(toks):
    rows, q = [], list(Q4)
    for t in toks:
        rows.append(list(q))
        q[t] = Fr(0)
        s = sum(q)
        q = [x / s for x in q] if s > 0 else q
    return rows


@pytest.mark.parametrize("k", [1, 2, 3])
def test_reading_of_algorithm1_preserves_target_without_replacement(k):
    """Distinct candidates, each with the distribution it was really drawn from (p_hat_i per candidate)."""
    total, total_bad = [Fr(0)] * 4, [Fr(0)] * 4
    for toks in itertools.permutations(range(4), k):
        rows = _without_replacement_rows(toks)
        w = Fr(1)
        for t, r in zip(toks, rows):
            w *= r[t]
        d = alg1_token_distribution(P4B, list(zip(toks, rows)))
        bad = alg1_token_distribution(P4B, [(t, Q4) for t in toks])  # wrong rows: must NOT give p
        total = [a + w * b for a, b in zip(total, d)]
        total_bad = [a + w * b for a, b in zip(total_bad, bad)]
    assert total == P4B
    if k > 1:
        assert total_bad != P4B


def test_scalar_reading_of_update_line_is_wrong():
    """Reading the garbled update as 'keep p, only touch the candidate token' breaks the guarantee,
    which is why the vector update of the Preliminaries is taken."""
    def scalar_variant(p, cands):
        p = list(p)
        reach, out = Fr(1), [Fr(0)] * len(p)
        for t, q in cands:
            a = min(Fr(1), p[t] / q[t])
            out[t] += reach * a
            reach *= 1 - a
            p[t] = max(Fr(0), p[t] - q[t])
            Z = sum(p)
            p = [x / Z for x in p]
        return [o + reach * x for o, x in zip(out, p)]
    total = [Fr(0)] * 4
    for t in range(4):
        d = scalar_variant(P4B, [(t, Q4)])
        total = [a + Q4[t] * b for a, b in zip(total, d)]
    assert total != P4B


# ----------------------------------------------------------- helpers to drive the C oracle

def _single_node_batch(p, rows, toks, uniforms_r, uniform_u, V):
    """One decision node: children of the context are the candidates; batch over uniform draws."""
    n = len(uniforms_r)
    k = len(toks)
    T = max(k, 1)
    target = np.zeros((n, T + 1, V), np.float32)
    target[:, 0] = np.array([float(x) for x in p], np.float32)
    target[:, 1:] = 1.0 / V
    draft = np.zeros((n, T, V), np.float32)
    for i, r in enumerate(rows):
        draft[:, i] = np.array([float(x) for x in r], np.float32)
    tokens = np.zeros((n, T), np.int32)
    tokens[:, :k] = np.array(toks, np.int32)
    parent = np.full((n, T), -1, np.int32)
    sizes = np.full((n,), k, np.int32)
    un = np.zeros((n, T + 1), np.float32)
    un[:, :k] = uniforms_r
    un[:, T] = uniform_u
    return target, draft, tokens, parent, un, sizes


def _first_token(res, tokens):
    """Token emitted first by each walk: the accepted child's token, else the final draw."""
    first = res["bonus_token"].copy()
    has = res["accept_len"] > 0
    idx = res["accepted_path"][:, 0]
    first[has] = tokens[np.arange(len(first))[has], idx[has]]
    return first


# --------------------------------------------------------- the C oracle against the exact model

def test_oracle_regions_match_exact_thresholds(oracle):
    """Probe each side of every decision boundary that the exact model predicts (V = 4, k = 2).
    All probabilities are multiples of 1/8, so fp32 inputs are exact."""
    toks = [1, 2]
    rows = [Q4, Q4]
    acc, reach, pf, thr = alg1_exact(P4, list(zip(toks, rows)))
    assert thr[0] == Fr(2, 3)           # p(1)/q(1) = (1/4)/(3/8)
    # after rejecting token 1: residual max(0,p-q) = (3/8,0,0,0) -> one-hot on token 0
    assert pf == [Fr(1), 0, 0, 0] and thr[1] == 0
    eps = 1e-4
    cases = [  # (r1, r2, u) -> expected first token
        ((float(thr[0]) - eps, 0.5, 0.5), 1),
        ((float(thr[0]) + eps, 0.0, 0.5), 0),      # token 2 has residual mass 0: never accepted
        ((float(thr[0]) + eps, 0.99, 0.99), 0),
        ((0.0, 0.0, 0.0), 1),
    ]
    r = np.array([[c[0][0], c[0][1]] for c in cases], np.float32)
    u = np.array([c[0][2] for c in cases], np.float32)
    t, d, tk, par, un, sz = _single_node_batch(P4, rows, toks, r, u, 4)
    res = oracle.tree_accept(t, d, tk, par, un, tree_sizes=sz)
    assert list(_first_token(res, tk)) == [c[1] for c in cases]


def test_oracle_final_draw_is_inverse_cdf(oracle):
    """k = 0 (a leaf): the final draw alone, cells of the CDF of p in ascending token id."""
    edges = np.cumsum([float(x) for x in P4])
    us, want = [], []
    lo = 0.0
    for v, hi in enumerate(edges):
        us += [lo + 1e-4, (lo + hi) / 2, hi - 1e-4]
        want += [v] * 3
        lo = hi
    n = len(us)
    t, d, tk, par, un, sz = _single_node_batch(P4, [], [], np.zeros((n, 0), np.float32), np.array(us, np.float32), 4)
    res = oracle.tree_accept(t, d, tk, par, un, tree_sizes=sz)
    assert list(res["bonus_token"]) == want and np.all(res["accept_len"] == 0)
    # u exactly on an edge belongs to the next cell (strict '>' in "cumsum > u*total")
    t, d, tk, par, un, sz = _single_node_batch(P4, [], [], np.zeros((2, 0), np.float32), np.array([0.5, 0.75], np.float32), 4)
    assert list(oracle.tree_accept(t, d, tk, par, un, tree_sizes=sz)["bonus_token"]) == [1, 2]


@pytest.mark.parametrize("toks,wr", [((2,), False), ((1, 0), False), ((3, 0, 1), True), ((0, 0), False)])
def test_oracle_monte_carlo_matches_exact_outcome(oracle, toks, wr):
    """Frequencies of the first emitted token over 2e5 uniform draws vs the exact model (5 sigma)."""
    n = 200_000
    rng = np.random.default_rng(1234 + len(toks))
    rows = _without_replacement_rows(toks) if wr else [Q4] * len(toks)
    exact = alg1_token_distribution(P4B, list(zip(toks, rows)))
    acc, reach, _, _ = alg1_exact(P4B, list(zip(toks, rows)))
    r = rng.random((n, len(toks)), dtype=np.float32)
    u = rng.random(n, dtype=np.float32)
    t, d, tk, par, un, sz = _single_node_batch(P4B, rows, list(toks), r, u, 4)
    res = oracle.tree_accept(t, d, tk, par, un, tree_sizes=sz)
    first = _first_token(res, tk)
    for v in range(4):
        pv = float(exact[v])
        sd = math.sqrt(max(pv * (1 - pv), 1e-12) / n)
        assert abs(np.mean(first == v) - pv) < 5 * sd + 1e-9
    # which candidate was accepted, and how often none was
    for i, a in enumerate(acc):
        f = np.mean((res["accept_len"] > 0) & (res["accepted_path"][:, 0] == i))
        assert abs(f - float(a)) < 5 * math.sqrt(max(float(a) * (1 - float(a)), 1e-12) / n) + 1e-9
    assert abs(np.mean(res["accept_len"] == 0) - float(reach)) < 5 * math.sqrt(0.25 / n)


def test_chain_is_classic_speculative_sampling(oracle):
    """Chain draft, one candidate per node (Preliminaries): P(accept) = sum_v min(p, p_hat) when the
    token is drawn from p_hat, emitted tokens follow (1 - a^(g+1)) / (1 - a), and the resampled token
    follows norm(max(0, p - p_hat))."""
    n, V, gamma = 100_000, 6, 4
    rng = np.random.default_rng(7)
    p = np.array([0.4, 0.3, 0.1, 0.1, 0.05, 0.05], np.float32)
    q = np.array([0.1, 0.2, 0.3, 0.2, 0.1, 0.1], np.float32)
    alpha = float(np.minimum(p.astype(np.float64), q.astype(np.float64)).sum())
    target = np.broadcast_to(p, (n, gamma + 1, V)).copy()
    draft = np.broadcast_to(q, (n, gamma, V)).copy()
    tokens = rng.choice(V, size=(n, gamma), p=q.astype(np.float64) / q.astype(np.float64).sum()).astype(np.int32)
    parent = np.broadcast_to(np.arange(-1, gamma - 1, dtype=np.int32), (n, gamma)).copy()
    un = rng.random((n, gamma + 1), dtype=np.float32)
    res = oracle.tree_accept(target, draft, tokens, parent, un)
    L = res["accept_len"]
    for j in range(gamma + 1):
        want = alpha ** j * (1 - alpha) if j < gamma else alpha ** gamma
        assert abs(np.mean(L == j) - want) < 5 * math.sqrt(want * (1 - want) / n)
    emitted = np.mean(L + 1)
    assert abs(emitted - (1 - alpha ** (gamma + 1)) / (1 - alpha)) < 0.02
    # paths are the chain prefix
    for j in range(gamma):
        assert np.all(res["accepted_path"][L > j, j] == j)
        assert np.all(res["accepted_path"][L <= j, j] == -1)
    # rejected at the first node => bonus ~ norm(max(0, p - q)), and never the rejected token's value
    rej = L == 0
    resid = np.maximum(p.astype(np.float64) - q.astype(np.float64), 0)
    resid /= resid.sum()
    counts = np.bincount(res["bonus_token"][rej], minlength=V)
    sup = resid > 0
    assert counts[~sup].sum() == 0
    chi = stats.chisquare(counts[sup], resid[sup] * counts.sum())
    assert chi.pvalue > 1e-3
    # all accepted => bonus ~ p
    full = L == gamma
    chi = stats.chisquare(np.bincount(res["bonus_token"][full], minlength=V), p.astype(np.float64) / p.astype(np.float64).sum() * full.sum())
    assert chi.pvalue > 1e-3


def test_degenerate_cases(oracle):
    V, T = 8, 3
    p = np.full((1, T + 1, V), 1.0 / V, np.float32)
    parent = np.array([[-1, 0, 1]], np.int32)
    tokens = np.array([[3, 5, 1]], np.int32)
    # p == p_hat: every candidate accepted whatever r < 1 is
    un = np.array([[0.999999, 0.5, 0.0, 0.3]], np.float32)
    res = oracle.tree_accept(p, p[:, :T].copy(), tokens, parent, un)
    assert list(res["accepted_path"][0]) == [0, 1, 2] and res["accept_len"][0] == 3
    assert res["bonus_token"][0] == 2  # u = 0.3 over 8 equal cells -> cell 2
    # disjoint supports: always rejected, residual = p, and the final draw comes from p itself
    pt = np.zeros((1, T + 1, V), np.float32)
    pt[:, :, :4] = 0.25
    qd = np.zeros((1, T, V), np.float32)
    qd[:, :, 4:] = 0.25
    tok = np.array([[5, 6, 7]], np.int32)
    res = oracle.tree_accept(pt, qd, tok, np.array([[-1, -1, -1]], np.int32), np.array([[0.0, 0.0, 0.0, 0.6]], np.float32))
    assert res["accept_len"][0] == 0 and res["bonus_token"][0] == 2 and res["n_sweeps"][0] == 4
    # r = 0 accepts iff p(t) > 0; p_hat(t) = 0 with p(t) > 0 accepts for every r
    qz = qd.copy()
    tok2 = np.array([[1, 6, 7]], np.int32)
    res = oracle.tree_accept(pt, qz, tok2, np.array([[-1, -1, -1]], np.int32), np.array([[0.99, 0, 0, 0.5]], np.float32))
    assert list(res["accepted_path"][0][:1]) == [0]
    # p <= p_hat everywhere after a rejection cannot happen with mass left; zero residual keeps p
    same = np.full((1, 2, V), 1.0 / V, np.float32)
    res = oracle.tree_accept(same, same[:, :1].copy(), np.array([[0]], np.int32), np.array([[-1]], np.int32),
                             np.array([[0.5, 0.9]], np.float32))
    assert res["accept_len"][0] == 1


def test_rejected_token_is_never_the_bonus_and_paths_are_valid(oracle):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=300, tree=(1, 12), vocab=40)
    inp = W.make_accept_inputs(cfg, salt=3, rho=0.5)
    res = oracle.tree_accept(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                             tree_sizes=inp.tree_sizes)
    par, tok = inp.tree_parent.numpy(), inp.draft_tokens.numpy()
    seen_reject = 0
    for b in range(cfg.batch):
        L = int(res["accept_len"][b])
        path = list(res["accepted_path"][b][:L])
        assert all(x == -1 for x in res["accepted_path"][b][L:])
        cur = -1
        for node in path:
            assert par[b, node] == cur and node < int(inp.tree_sizes[b])
            cur = node
        kids = [i for i in range(int(inp.tree_sizes[b])) if par[b, i] == cur]
        # all children of the last node were rejected: none of their tokens can be drawn afterwards
        seen_reject += len(kids)
        assert int(res["bonus_token"][b]) not in {int(tok[b, i]) for i in kids}
        assert res["n_sweeps"][b] >= 1 + len(kids)
    assert seen_reject > 100


# ------------------------------------------------------------------------------------- greedy

def test_greedy_equals_stochastic_rule_on_one_hot_targets(oracle):
    """Temperature 0 makes the target one-hot at its argmax; Algorithm 1 on that one-hot row must walk
    the same path and emit the same token as the argmax-match rule."""
    cfg = W.scaled(W.CONFIGS["tiny"], batch=200, tree=(1, 10), vocab=12)
    inp = W.make_accept_inputs(cfg, salt=5, rho=0.9, greedy="all", rho_greedy=0.9)
    tp = inp.target_probs.numpy()
    onehot = np.zeros_like(tp)
    np.put_along_axis(onehot, tp.argmax(-1)[..., None], 1.0, axis=-1)
    # draft rows must give the candidate token positive probability for the ratio test to be defined
    g = oracle.tree_accept(tp, None, inp.draft_tokens, inp.tree_parent, None, tree_sizes=inp.tree_sizes,
                           greedy=np.ones(cfg.batch, np.uint8))
    s = oracle.tree_accept(onehot, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                           tree_sizes=inp.tree_sizes)
    assert np.array_equal(g["accepted_path"], s["accepted_path"])
    assert np.array_equal(g["bonus_token"], s["bonus_token"])
    assert g["accept_len"].max() >= 2


def test_greedy_is_longest_argmax_match_brute_force(oracle):
    rng = np.random.default_rng(11)
    V, T = 5, 6
    for _ in range(200):
        parent = np.array([[rng.integers(-1, i) for i in range(T)]], np.int32)
        tokens = rng.integers(0, V, size=(1, T)).astype(np.int32)
        tp = rng.random((1, T + 1, V)).astype(np.float32)
        res = oracle.tree_accept(tp, None, tokens, parent, None, greedy=np.ones(1, np.uint8))
        cur, path = -1, []
        while True:
            a = int(np.argmax(tp[0, cur + 1]))
            nxt = [i for i in range(T) if parent[0, i] == cur and tokens[0, i] == a]
            if not nxt:
                break
            cur = nxt[0]
            path.append(cur)
        assert list(res["accepted_path"][0][:len(path)]) == path and res["accept_len"][0] == len(path)
        assert res["bonus_token"][0] == a
    # ties: lowest token id wins
    tp = np.full((1, 2, 4), 0.25, np.float32)
    res = oracle.tree_accept(tp, None, np.array([[0]], np.int32), np.array([[-1]], np.int32), None,
                             greedy=np.ones(1, np.uint8))
    assert res["accept_len"][0] == 1 and res["bonus_token"][0] == 0


# ------------------------------------------------------------------------- distribution (chi-square)

def test_output_distribution_matches_target_chi_square(oracle):
    """16-token vocabulary, first-order Markov target, tree = 3 children of the context x 2 children each,
    draft tokens re-drawn from their draft rows in every trial: the first emitted token must follow
    the context row and the second, given the first, the Markov row (Sec. 3.3: the output distribution
    equals the target's)."""
    V, n = 16, 120_000
    rng = np.random.default_rng(2024)
    p_root = rng.dirichlet(np.ones(V)).astype(np.float32)
    P2 = rng.dirichlet(np.ones(V), size=V).astype(np.float32)
    q_root = rng.dirichlet(np.ones(V)).astype(np.float32)
    Q2 = rng.dirichlet(np.ones(V), size=V).astype(np.float32)
    parent1 = np.array([-1, -1, -1, 0, 0, 1, 1, 2, 2], np.int32)
    T = len(parent1)
    parent = np.broadcast_to(parent1, (n, T)).copy()
    tokens = np.zeros((n, T), np.int32)
    cdf_root = np.cumsum(q_root.astype(np.float64) / q_root.astype(np.float64).sum())
    tokens[:, :3] = np.searchsorted(cdf_root, rng.random((n, 3)), side="right").clip(0, V - 1)
    cdf2 = np.cumsum(Q2.astype(np.float64) / Q2.astype(np.float64).sum(1, keepdims=True), axis=1)
    for i in range(3, T):
        par_tok = tokens[:, parent1[i]]
        tokens[:, i] = (rng.random(n)[:, None] > cdf2[par_tok]).sum(1).clip(0, V - 1)
    target = np.zeros((n, T + 1, V), np.float32)
    target[:, 0] = p_root
    draft = np.zeros((n, T, V), np.float32)
    draft[:, :3] = q_root
    for i in range(T):
        target[:, i + 1] = P2[tokens[:, i]]
        if i >= 3:
            draft[:, i] = Q2[tokens[:, parent1[i]]]
    un = rng.random((n, T + 1), dtype=np.float32)
    res = oracle.tree_accept(target, draft, tokens, parent, un)
    L, path, bonus = res["accept_len"], res["accepted_path"], res["bonus_token"]
    rows = np.arange(n)
    first = np.where(L > 0, tokens[rows, np.maximum(path[:, 0], 0)], bonus)
    pr = p_root.astype(np.float64) / p_root.astype(np.float64).sum()
    chi1 = stats.chisquare(np.bincount(first, minlength=V), pr * n)
    assert chi1.pvalue > 1e-3, chi1
    has2 = L > 0
    second = np.where(L > 1, tokens[rows, np.maximum(path[:, 1], 0)], bonus)
    pvals = []
    for x in range(V):
        sel = has2 & (first == x)
        if sel.sum() < 2000:
            continue
        px = P2[x].astype(np.float64) / P2[x].astype(np.float64).sum()
        pvals.append(stats.chisquare(np.bincount(second[sel], minlength=V), px * sel.sum()).pvalue)
    assert len(pvals) >= 8 and min(pvals) > 1e-4, pvals
    # negative control: the same test must fail when tokens are NOT re-drawn (fixed tree, fresh uniforms)
    tokens_fixed = np.broadcast_to(tokens[0], (n, T)).copy()
    target_f = np.broadcast_to(target[0], target.shape).copy()
    draft_f = np.broadcast_to(draft[0], draft.shape).copy()
    res_f = oracle.tree_accept(target_f, draft_f, tokens_fixed, parent, un)
    first_f = np.where(res_f["accept_len"] > 0, tokens_fixed[rows, np.maximum(res_f["accepted_path"][:, 0], 0)],
                       res_f["bonus_token"])
    assert stats.chisquare(np.bincount(first_f, minlength=V), pr * n).pvalue < 1e-6
    assert 1.0 < (L + 1).mean() < 3.0


# ------------------------------------------------------------------------------ workload statistic

def test_gaussian_logit_acceptance_rate_closed_form():
    """i.i.d. N(0, variance 2) logits: E[sum_v min(p, p_hat)] = 2*Phi(-sigma/sqrt(2)) = 0.3173; this is the
    per-candidate acceptance rate of the rho = 0 synthetic workload."""
    cfg = W.scaled(W.CONFIGS["7b_mha"], batch=2, tree=(3, 3))
    inp = W.make_accept_inputs(cfg, rho=0.0)
    t = inp.target_probs[:, 0].double()
    d = inp.draft_probs[:, 0].double()
    m = torch_min_sum(t, d)
    assert abs(m - 2 * stats.norm.cdf(-1.0)) < 0.02


def torch_min_sum(t, d):
    import torch
    return float(torch.minimum(t, d).sum(-1).mean())


def test_margins_reported(oracle):
    t, d, tk, par, un, sz = _single_node_batch(P4, [Q4], [1], np.array([[0.5]], np.float32), np.array([0.1], np.float32), 4)
    res = oracle.tree_accept(t, d, tk, par, un, tree_sizes=sz)
    # accept test margin |0.5 - 2/3|; then the child is a leaf with a uniform row: u = 0.1 in cell [0, .25)
    assert res["accept_len"][0] == 1
    assert abs(res["min_margin"][0] - 0.1) < 1e-6


def test_worked_example_fixture(oracle):
    """Hand-derived thresholds of Algorithm 1 on a 4-token example (tests/golden/alg1_worked_example.txt)."""
    import os
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "alg1_worked_example.txt"))
            if l.strip() and not l.startswith("#")]
    r = np.array([[float(x) for x in row[:3]] for row in rows], np.float32)
    u = np.array([float(row[3]) for row in rows], np.float32)
    want = [int(row[4]) for row in rows]
    toks = [1, 3, 2]
    # the fixture's thresholds are also what the exact model gives
    _, _, pf, thr = alg1_exact(P4B, [(t, Q4) for t in toks])
    assert thr == [Fr(1, 3), Fr(0), Fr(8, 15)] and pf == [Fr(1), 0, 0, 0]
    t, d, tk, par, un, sz = _single_node_batch(P4B, [Q4] * 3, toks, r, u, 4)
    res = oracle.tree_accept(t, d, tk, par, un, tree_sizes=sz)
    assert list(_first_token(res, tk)) == want


# --------------------------------------------------------- the decision trace (what the parity tests classify mismatches with)

def test_trace_of_worked_example(oracle):
    """The decisions of the hand-derived example, one by one: kinds, nodes and margins follow from its thresholds
    (1/3, 0, 8/15) and from the final distributions (one-hot on token 0 at the context; uniform at an accepted leaf)."""
    toks = [1, 3, 2]
    r = np.array([[0.3333, 0.9, 0.9], [0.3334, 0.0, 0.5333], [0.3334, 0.0, 0.5334]], np.float32)
    u = np.array([0.9, 0.5, 0.0], np.float32)
    t, d, tk, par, un, sz = _single_node_batch(P4B, [Q4] * 3, toks, r, u, 4)
    res = oracle.tree_accept(t, d, tk, par, un, tree_sizes=sz)
    A, R, B = oracle.DEC_ACCEPT, oracle.DEC_REJECT, oracle.DEC_BONUS
    want = [
        # accepted at once; node 0 is then a leaf whose row is uniform: u = 0.9 lies in cell [0.75, 1)
        [(A, 0, abs(float(r[0, 0]) - 1 / 3)), (B, 0, 0.1)],
        # first rejected; second has residual mass 0 (ratio 0, r = 0: on the boundary); third accepted; leaf: u = 0.5 on an edge
        [(R, 0, abs(float(r[1, 0]) - 1 / 3)), (R, 1, 0.0), (A, 2, abs(float(r[1, 2]) - 8 / 15)), (B, 2, 0.0)],
        # all three rejected: final draw at the context from a one-hot distribution, u = 0 on the lower edge
        [(R, 0, abs(float(r[2, 0]) - 1 / 3)), (R, 1, 0.0), (R, 2, abs(float(r[2, 2]) - 8 / 15)), (B, -1, 0.0)],
    ]
    for b, decs in enumerate(want):
        assert res["n_dec"][b] == len(decs)
        for j, (kind, node, margin) in enumerate(decs):
            assert (res["dec_kind"][b, j], res["dec_node"][b, j]) == (kind, node), (b, j)
            assert abs(res["dec_margin"][b, j] - margin) < 1e-6, (b, j, res["dec_margin"][b, j], margin)
        assert abs(res["min_margin"][b] - min(m for _, _, m in decs)) < 1e-6


def _replay(oracle_mod, res, b, parent):
    """Path and 'a final draw / argmax ended the walk' rebuilt from the decision list alone."""
    path, cur = [], -1
    for j in range(int(res["n_dec"][b])):
        kind, node = int(res["dec_kind"][b, j]), int(res["dec_node"][b, j])
        if kind in (oracle_mod.DEC_ACCEPT, oracle_mod.DEC_REJECT):
            assert int(parent[node]) == cur            # a candidate is a child of the current node
            if kind == oracle_mod.DEC_ACCEPT:
                path.append(node)
                cur = node
        elif kind == oracle_mod.DEC_BONUS:
            assert node == cur and j == int(res["n_dec"][b]) - 1
        else:
            assert node == cur
            if j + 1 < int(res["n_dec"][b]):           # not the last argmax: it matched a child
                nxt = int(res["dec_node"][b, j + 1])
                assert int(parent[nxt]) == cur
                path.append(nxt)
                cur = nxt
    return path


def test_trace_replays_to_the_result_and_tolerance_helper_finds_first_difference(oracle):
    from oracle.compare import first_differing_decision, compare_with_oracle
    cfg = W.scaled(W.CONFIGS["tiny"], batch=40, tree=(3, 30), max_depth=6, vocab=50)
    inp = W.make_accept_inputs(cfg, salt=5, rho=0.9, greedy="half")
    res = oracle.tree_accept(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                             tree_sizes=inp.tree_sizes, greedy=inp.greedy)
    par = inp.tree_parent.numpy()
    T = cfg.max_tree
    flipped = 0
    for b in range(cfg.batch):
        n = int(res["n_dec"][b])
        assert 1 <= n <= T + 1
        path = _replay(oracle, res, b, par[b])
        assert path == [int(x) for x in res["accepted_path"][b] if x >= 0]
        finite = res["dec_margin"][b, :n]
        assert np.isclose(finite.min(), res["min_margin"][b]) or (np.isinf(finite.min()) and np.isinf(res["min_margin"][b]))
        # identical outputs contradict no decision
        assert first_differing_decision(res, b, res["accepted_path"][b], res["bonus_token"][b]) is None
        if inp.greedy[b]:
            continue
        # pretend the other side took decision j the other way, for every accept test j: the helper must point at j
        for j in range(n):
            kind, node = int(res["dec_kind"][b, j]), int(res["dec_node"][b, j])
            depth = sum(1 for i in range(j) if res["dec_kind"][b, i] == oracle.DEC_ACCEPT)
            fake = res["accepted_path"][b].copy()
            if kind == oracle.DEC_ACCEPT:
                fake[depth:] = -1                                  # it rejected the candidate and every later one
            elif kind == oracle.DEC_REJECT:
                fake[depth:] = -1
                fake[depth] = node                                 # it accepted the candidate and stopped there
            else:
                continue
            assert first_differing_decision(res, b, fake, (int(res["bonus_token"][b]) + 1) % cfg.vocab) == j
            flipped += 1
        fake_bonus = (int(res["bonus_token"][b]) + 1) % cfg.vocab   # same path, another final draw: the last decision
        assert first_differing_decision(res, b, res["accepted_path"][b], fake_bonus) == n - 1
    assert flipped > 50
    # the tolerance applies at the first differing decision only
    b = next(b for b in range(cfg.batch) if not inp.greedy[b] and res["accept_len"][b] >= 1)
    path, bonus, alen = res["accepted_path"].copy(), res["bonus_token"].copy(), res["accept_len"].copy()
    path[b, :] = -1
    alen[b] = 0
    with pytest.raises(AssertionError):
        compare_with_oracle(res, path, bonus, alen, inp.greedy)      # a wrong decision far from its boundary
    d = first_differing_decision(res, b, path[b], bonus[b])
    res2 = {k: v.copy() for k, v in res.items()}
    res2["dec_margin"][b, d] = 1e-7
    assert compare_with_oracle(res2, path, bonus, alen, inp.greedy) == 1
