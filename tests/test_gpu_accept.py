"""Parity of the CUDA acceptance kernel (through the C ABI) with the oracle's walk.  Needs a B200.

Greedy sequences must agree exactly.  Stochastic sequences must agree exactly given the same uniforms,
except where the oracle's margin at the FIRST decision that differs is below 1e-5 (the decisions are
compared one by one, see oracle/compare.py); such sequences are counted, and the count is asserted to stay small.
"""
import os

import numpy as np
import pytest
import torch
from scipy import stats

from oracle.compare import compare_with_oracle
from paper_2401_15077_b200 import workloads as W

pytestmark = pytest.mark.gpu

SALTS = int(os.environ.get("EAGLE_ACCEPT_SALTS", "3"))   # seeds per case (more for a longer soak)
MARGIN = 1e-5


@pytest.fixture(scope="module")
def E():
    from paper_2401_15077_b200 import build, binding
    build.build()
    binding.load()
    assert torch.cuda.is_available()
    return binding


def _gpu_accept(E, inp, greedy_flags=True, path_cap=None, draft=True):
    d = torch.device("cuda:0")
    B = inp.target_probs.shape[0]
    status = torch.zeros(1, dtype=torch.int32, device=d)
    alen = torch.full((B,), -7, dtype=torch.int32, device=d)
    path, bonus = E.eagle_tree_accept(inp.target_probs.to(d), inp.draft_probs.to(d) if draft else None,
                                      inp.draft_tokens.to(d), inp.tree_parent.to(d),
                                      inp.uniforms.to(d) if draft else None, tree_sizes=inp.tree_sizes.to(d),
                                      greedy=inp.greedy.to(d) if greedy_flags else None, accept_len=alen,
                                      status=status, path_cap=path_cap)
    torch.cuda.synchronize()
    return path.cpu().numpy(), bonus.cpu().numpy(), alen.cpu().numpy(), int(status.item())


def _compare(inp, ref, path, bonus, alen):
    """Returns the number of tolerated (near-boundary at the first differing decision) mismatches; asserts on any other."""
    return compare_with_oracle(ref, path, bonus, alen, inp.greedy.numpy(), MARGIN)


CASES = [
    ("tiny", W.CONFIGS["tiny"], dict(rho=0.9), "none"),
    ("tiny_greedy", W.CONFIGS["tiny"], dict(rho=0.9, greedy="all"), "all"),
    ("tiny_rho0", W.CONFIGS["tiny"], dict(rho=0.0), "none"),
    ("7b_t1", W.CONFIGS["7b_mha"], dict(rho=0.9), "none"),
    ("7b_t0", W.CONFIGS["7b_mha"], dict(rho=0.9, greedy="all"), "all"),
    ("70b", W.CONFIGS["70b_gqa"], dict(rho=0.9), "none"),
    ("70b_rho0", W.CONFIGS["70b_gqa"], dict(rho=0.0), "none"),
    ("mix_small", W.scaled(W.CONFIGS["serving_mix"], batch=12), dict(rho=0.9), "half"),
    ("odd_vocab_batch", W.scaled(W.CONFIGS["tiny"], batch=300, tree=(0, 20), vocab=4099), dict(rho=0.7, greedy="half"), "half"),
    ("small_vocab_batch", W.scaled(W.CONFIGS["tiny"], batch=2000, tree=(0, 14), vocab=37), dict(rho=0.5, greedy="half"), "half"),
]


# Batch sizes that land on every team layout of the large-vocabulary kernel: clusters of 8, 4, 2 and single CTAs
# (the launcher picks the widest cluster that keeps at most four CTAs per SM).
WIDTH_CASES = [(8, 20), (4, 100), (2, 200), (1, 640)]


@pytest.mark.parametrize("width,batch", WIDTH_CASES, ids=[f"cluster{w}" for w, _ in WIDTH_CASES])
@pytest.mark.parametrize("logits", [False, True], ids=["probs", "logits"])
def test_every_cluster_width_matches_oracle(E, oracle, width, batch, logits):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=batch, tree=(1, 16), max_depth=5, vocab=8192)
    # the library says which layout this call gets on this GPU (148 SMs: up to 74 / 148 / 296 trees for 8 / 4 / 2 CTAs)
    assert E.eagle_tree_accept_cluster_width(batch, cfg.vocab) == width
    assert E.eagle_tree_accept_cluster_width(batch, 4096) == 0
    inp = W.make_accept_inputs(cfg, salt=width, rho=0.85, greedy="half", logits=logits)
    d = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=d)
    alen = torch.full((batch,), -7, dtype=torch.int32, device=d)
    args = (inp.target_probs.to(d), inp.draft_probs.to(d), inp.draft_tokens.to(d), inp.tree_parent.to(d), inp.uniforms.to(d))
    kw = dict(tree_sizes=inp.tree_sizes.to(d), greedy=inp.greedy.to(d), accept_len=alen, status=status)
    if logits:
        ref = oracle.tree_accept_logits(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms, 0.9,
                                        tree_sizes=inp.tree_sizes, greedy=inp.greedy)
        path, bonus = E.eagle_tree_accept_logits(*args, 0.9, **kw)
    else:
        ref = oracle.tree_accept(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                                 tree_sizes=inp.tree_sizes, greedy=inp.greedy)
        path, bonus = E.eagle_tree_accept(*args, **kw)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert _compare(inp, ref, path.cpu().numpy(), bonus.cpu().numpy(), alen.cpu().numpy()) <= max(1, batch // 100)
    assert int(ref["accept_len"].sum()) > batch // 4 and int((ref["n_sweeps"] > 2).sum()) > batch // 10   # the walks went somewhere


def test_full_size_serving_mix_matches_oracle(E, oracle):
    """The batched configuration at its full size (64 trees, vocabulary 32000, half greedy): clusters of eight in two waves."""
    cfg = W.CONFIGS["serving_mix"]
    inp = W.make_accept_inputs(cfg, salt=0, rho=0.9)
    assert E.eagle_tree_accept_cluster_width(cfg.batch, cfg.vocab) == 8
    ref = oracle.tree_accept(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                             tree_sizes=inp.tree_sizes, greedy=inp.greedy)
    path, bonus, alen, status = _gpu_accept(E, inp)
    assert status == 0
    assert _compare(inp, ref, path, bonus, alen) <= 1
    assert int(ref["accept_len"].sum()) > cfg.batch


def test_all_greedy_call_without_draft_rows_takes_clusters_of_four(E, oracle):
    """Temperature 0 for the whole batch, no draft rows and no uniforms passed: at 64 trees clusters of eight would need a
    second wave, so this kind of call takes four CTAs per tree; the tokens are the oracle's exactly."""
    cfg = W.CONFIGS["serving_mix"]
    inp = W.make_accept_inputs(cfg, salt=3, greedy="all")
    assert inp.greedy.all()
    assert E.eagle_tree_accept_cluster_width(cfg.batch, cfg.vocab, all_greedy=True) == 4
    assert E.eagle_tree_accept_cluster_width(20, cfg.vocab, all_greedy=True) == 8
    assert E.eagle_tree_accept_cluster_width(100, cfg.vocab, all_greedy=True) == 4      # (as for any call of that size)
    ref = oracle.tree_accept(inp.target_probs, None, inp.draft_tokens, inp.tree_parent, None, tree_sizes=inp.tree_sizes, greedy=inp.greedy)
    path, bonus, alen, status = _gpu_accept(E, inp, draft=False)
    assert status == 0
    assert _compare(inp, ref, path, bonus, alen) == 0
    assert int(ref["accept_len"].sum()) > cfg.batch
    # the same batch with the draft rows passed (clusters of eight): the same tokens
    path8, bonus8, alen8, status = _gpu_accept(E, inp)
    assert status == 0 and np.array_equal(path, path8) and np.array_equal(bonus, bonus8) and np.array_equal(alen, alen8)


@pytest.mark.parametrize("name,cfg,kw,mode", CASES, ids=[c[0] for c in CASES])
def test_accept_matches_oracle(E, oracle, name, cfg, kw, mode):
    tolerated_total, seqs = 0, 0
    for salt in range(SALTS if cfg.batch * cfg.vocab < 4_000_000 else max(1, SALTS // 3)):
        inp = W.make_accept_inputs(cfg, salt=salt, **kw)
        ref = oracle.tree_accept(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                                 tree_sizes=inp.tree_sizes, greedy=inp.greedy)
        path, bonus, alen, status = _gpu_accept(E, inp)
        assert status == 0
        tolerated_total += _compare(inp, ref, path, bonus, alen)
        seqs += cfg.batch
    # near-boundary disagreements are possible in principle, but fp64 sums make them very rare
    assert tolerated_total <= max(1, seqs // 100), tolerated_total


LOGIT_CASES = [
    ("tiny_t1", W.CONFIGS["tiny"], dict(rho=0.9), 1.0),
    ("tiny_half_greedy_t07", W.CONFIGS["tiny"], dict(rho=0.9, greedy="half"), 0.7),
    ("7b_t1", W.CONFIGS["7b_mha"], dict(rho=0.9), 1.0),
    ("70b_t13", W.CONFIGS["70b_gqa"], dict(rho=0.9), 1.3),
    ("70b_rho0", W.CONFIGS["70b_gqa"], dict(rho=0.0), 1.0),
    ("mix_small_t08", W.scaled(W.CONFIGS["serving_mix"], batch=12), dict(rho=0.9), 0.8),
    ("odd_vocab_batch", W.scaled(W.CONFIGS["tiny"], batch=300, tree=(0, 20), vocab=4099), dict(rho=0.7, greedy="half"), 1.0),
    ("small_vocab_batch", W.scaled(W.CONFIGS["tiny"], batch=2000, tree=(0, 14), vocab=37), dict(rho=0.5, greedy="half"), 0.5),
]


@pytest.mark.parametrize("name,cfg,kw,temperature", LOGIT_CASES, ids=[c[0] for c in LOGIT_CASES])
def test_accept_on_logits_matches_oracle(E, oracle, name, cfg, kw, temperature):
    """eagle_tree_accept_logits against the oracle's fp64 softmax walk.  The kernel's exponentials are fp32, so a
    decision may differ where the oracle's margin is below 1e-5; such sequences are counted."""
    tolerated_total, seqs, accepted = 0, 0, 0
    d = torch.device("cuda:0")
    for salt in range(SALTS if cfg.batch * cfg.vocab < 4_000_000 else max(1, SALTS // 3)):
        inp = W.make_accept_inputs(cfg, salt=salt, logits=True, **kw)
        ref = oracle.tree_accept_logits(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                                        temperature, tree_sizes=inp.tree_sizes, greedy=inp.greedy)
        status = torch.zeros(1, dtype=torch.int32, device=d)
        alen = torch.full((cfg.batch,), -7, dtype=torch.int32, device=d)
        path, bonus = E.eagle_tree_accept_logits(inp.target_probs.to(d), inp.draft_probs.to(d), inp.draft_tokens.to(d),
                                                 inp.tree_parent.to(d), inp.uniforms.to(d), temperature,
                                                 tree_sizes=inp.tree_sizes.to(d), greedy=inp.greedy.to(d), accept_len=alen,
                                                 status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        tolerated_total += _compare(inp, ref, path.cpu().numpy(), bonus.cpu().numpy(), alen.cpu().numpy())
        seqs += cfg.batch
        accepted += int(ref["accept_len"].sum())
    assert accepted >= 1        # the walks went somewhere (a single short sequence may accept nothing under one seed)
    assert tolerated_total <= max(1, seqs // 50), tolerated_total


def test_accept_on_logits_rejects_bad_temperature(E):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=2, vocab=64)
    inp = W.make_accept_inputs(cfg, logits=True)
    d = torch.device("cuda:0")
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(Exception):
            E.eagle_tree_accept_logits(inp.target_probs.to(d), inp.draft_probs.to(d), inp.draft_tokens.to(d), inp.tree_parent.to(d),
                                       inp.uniforms.to(d), bad)


def test_all_greedy_without_draft_rows(E, oracle):
    cfg = W.scaled(W.CONFIGS["7b_mha"], batch=3)
    inp = W.make_accept_inputs(cfg, salt=9, greedy="all")
    ref = oracle.tree_accept(inp.target_probs, None, inp.draft_tokens, inp.tree_parent, None, tree_sizes=inp.tree_sizes,
                             greedy=inp.greedy)
    path, bonus, alen, status = _gpu_accept(E, inp, draft=False)
    assert status == 0
    assert _compare(inp, ref, path, bonus, alen) == 0
    assert ref["accept_len"].max() >= 1


def test_path_cap_and_full_width_tree(E, oracle):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=40, tree=(64, 64), max_depth=64, vocab=50)
    inp = W.make_accept_inputs(cfg, salt=1, rho=0.95)
    ref = oracle.tree_accept(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                             tree_sizes=inp.tree_sizes, path_cap=70)
    path, bonus, alen, status = _gpu_accept(E, inp, greedy_flags=False, path_cap=70)
    assert status == 0 and path.shape == (40, 70)
    assert _compare(inp, ref, path, bonus, alen) <= 1


def test_invalid_inputs_are_reported(E):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=4, vocab=64)
    inp = W.make_accept_inputs(cfg, salt=2)
    inp.draft_tokens[1, 0] = 64        # outside the vocabulary
    inp.tree_parent[2, 3] = 5          # parent after child
    path, bonus, alen, status = _gpu_accept(E, inp)
    assert status in (-5, -7)
    assert bonus[1] == -1 and bonus[2] == -1 and alen[1] == 0 and alen[2] == 0
    assert (path[1] == -1).all() and (path[2] == -1).all()
    assert bonus[0] >= 0 and bonus[3] >= 0


def test_output_distribution_on_gpu_chi_square(E):
    """The kernel itself preserves the target distribution (Sec. 3.3): 16-token vocabulary, 3 children of the
    context, tokens re-drawn per trial, one batched call of 1e5 trees."""
    V, n = 16, 100_000
    rng = np.random.default_rng(99)
    p_root = rng.dirichlet(np.ones(V)).astype(np.float32)
    q_root = rng.dirichlet(np.ones(V)).astype(np.float32)
    T = 3
    cdf = np.cumsum(q_root.astype(np.float64) / q_root.astype(np.float64).sum())
    tokens = np.searchsorted(cdf, rng.random((n, T)), side="right").clip(0, V - 1).astype(np.int32)
    target = np.broadcast_to(p_root, (n, T + 1, V)).copy()
    draft = np.broadcast_to(q_root, (n, T, V)).copy()
    parent = np.full((n, T), -1, np.int32)
    un = rng.random((n, T + 1), dtype=np.float32)
    d = torch.device("cuda:0")
    alen = torch.zeros(n, dtype=torch.int32, device=d)
    path, bonus = E.eagle_tree_accept(torch.from_numpy(target).to(d), torch.from_numpy(draft).to(d),
                                      torch.from_numpy(tokens).to(d), torch.from_numpy(parent).to(d),
                                      torch.from_numpy(un).to(d), accept_len=alen)
    torch.cuda.synchronize()
    path, bonus, alen = path.cpu().numpy(), bonus.cpu().numpy(), alen.cpu().numpy()
    first = np.where(alen > 0, tokens[np.arange(n), np.maximum(path[:, 0], 0)], bonus)
    pr = p_root.astype(np.float64) / p_root.astype(np.float64).sum()
    assert stats.chisquare(np.bincount(first, minlength=V), pr * n).pvalue > 1e-3


@pytest.mark.parametrize("ragged", [True, False])
def test_host_step_entry_matches_device_calls(E, ragged):
    """eagle_tree_verify_step_host (copies in, attention, acceptance, copies out) gives what the two device calls give.
    Ragged lengths take the sequence-by-sequence copies of the visible slots and existing rows only (the arena is filled
    with NaN bit patterns first: nothing that was not copied may be read); equal full-size sequences take whole-tensor copies."""
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=5, prefix=(50, 900) if ragged else (700, 700), tree=(16, 64) if ragged else (64, 64),
                   max_depth=12, vocab=3000)
    attn = W.make_attn_inputs(cfg, salt=3)
    acc = W.make_accept_inputs(cfg, salt=3, trees=(attn.tree_sizes, attn.tree_parent))
    d = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=d)
    out = E.eagle_tree_verify_attn(attn.q.to(d), attn.k_cache.to(d), attn.v_cache.to(d), attn.seq_lens.to(d),
                                   attn.tree_parent.to(d), tree_sizes=attn.tree_sizes.to(d), status=status)
    path, bonus, alen, st = _gpu_accept(E, acc)
    host = dict(q=attn.q, k_cache=attn.k_cache, v_cache=attn.v_cache, seq_lens=attn.seq_lens, tree_sizes=attn.tree_sizes,
                tree_parent=attn.tree_parent, target_probs=acc.target_probs, draft_probs=acc.draft_probs,
                draft_tokens=acc.draft_tokens, uniforms=acc.uniforms, greedy=acc.greedy)
    runner = E.HostStepRunner({k: v.pin_memory() for k, v in host.items()}, d)
    assert (runner.h2d_bytes < runner.full_h2d_bytes) == ragged
    runner.arena.fill_(255)
    for _ in range(2):
        runner.run()
        torch.cuda.synchronize()
        assert int(runner.status.item()) == 0 and st == 0 and int(status.item()) == 0
        assert torch.equal(runner.out.view(torch.int16), out.cpu().view(torch.int16))
        assert np.array_equal(runner.accepted_path.numpy(), path) and np.array_equal(runner.bonus_token.numpy(), bonus)
        assert np.array_equal(runner.accept_len.numpy(), alen)


@pytest.mark.parametrize("mode", ["none", "half"])
def test_one_tree_shared_by_every_sequence(E, oracle, mode):
    """tree_parent given once ([T_max]) for all sequences: same tokens as the call that repeats it per sequence."""
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=10, vocab=5000)
    sizes, parent = W.make_trees(cfg, 3)
    n0 = int(sizes.max())
    row = parent[int(sizes.argmax())]
    trees = (torch.full((cfg.batch,), n0, dtype=torch.int32), row[None, :].expand(cfg.batch, -1).contiguous())
    inp = W.make_accept_inputs(cfg, salt=3, trees=trees, greedy=mode)
    ref = oracle.tree_accept(inp.target_probs, inp.draft_probs, inp.draft_tokens, inp.tree_parent, inp.uniforms,
                             tree_sizes=inp.tree_sizes, greedy=inp.greedy)
    d = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=d)
    alen = torch.full((cfg.batch,), -7, dtype=torch.int32, device=d)
    path, bonus = E.eagle_tree_accept(inp.target_probs.to(d), inp.draft_probs.to(d), inp.draft_tokens.to(d), row.contiguous().to(d),
                                      inp.uniforms.to(d), tree_sizes=trees[0][:1].to(d), greedy=inp.greedy.to(d), accept_len=alen,
                                      status=status, shared_tree=True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert _compare(inp, ref, path.cpu().numpy(), bonus.cpu().numpy(), alen.cpu().numpy()) == 0
    assert int(alen.sum()) > 0
