"""Parity of the CUDA tree attention (through the C ABI) with the fp64 oracle.  Needs a B200."""
import os

import numpy as np
import pytest
import torch

from paper_2401_15077_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3   # unit-variance bf16 inputs: bounds on |gpu - oracle|


@pytest.fixture(scope="module")
def E():
    from paper_2401_15077_b200 import build, binding
    build.build()
    binding.load()
    assert torch.cuda.is_available()
    return binding


def _to_dev(inp):
    d = torch.device("cuda:0")
    return dict(q=inp.q.to(d), k=inp.k_cache.to(d), v=inp.v_cache.to(d), sl=inp.seq_lens.to(d),
                par=inp.tree_parent.to(d), ts=inp.tree_sizes.to(d))


def _run(E, inp, num_splits=0, use_sizes=True, sm_scale=0.0):
    t = _to_dev(inp)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    out = torch.full_like(t["q"], float("nan"))
    E.eagle_tree_verify_attn(t["q"], t["k"], t["v"], t["sl"], t["par"], out, tree_sizes=t["ts"] if use_sizes else None,
                             num_splits=num_splits, status=status, sm_scale=sm_scale)
    torch.cuda.synchronize()
    return out.cpu(), int(status.item())


def _check(out, ref, sizes):
    got = out.double().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - ref)
    rows = np.zeros(ref.shape[:2], bool)
    for b, n in enumerate(sizes):
        rows[b, :int(n)] = True
        assert np.all(got[b, int(n):] == 0.0), "rows past the tree size must be zero"
    if rows.any():
        assert err[rows].max() <= MAX_ABS, err[rows].max()
        assert err[rows].mean() <= MEAN_ABS, err[rows].mean()
    return float(err.max())


CASES = {
    "tiny": W.CONFIGS["tiny"],
    "7b_mha": W.CONFIGS["7b_mha"],
    "70b_gqa": W.CONFIGS["70b_gqa"],
    "mixtral_gqa_small": W.scaled(W.CONFIGS["mixtral_gqa"], batch=2, prefix=(1500, 3000)),
    "serving_mix_small": W.scaled(W.CONFIGS["serving_mix"], batch=6, prefix=(100, 1500)),
    "d64_gqa_ragged": W.scaled(W.CONFIGS["tiny"], batch=5, num_q_heads=16, num_kv_heads=4, prefix=(0, 700), tree=(1, 33)),
    # group sizes that do not divide 128: the query tile is staged by the softmax threads instead of TMA
    "group3_d128": W.scaled(W.CONFIGS["7b_mha"], batch=3, num_q_heads=12, num_kv_heads=4, prefix=(50, 1200), tree=(3, 64), max_depth=8),
    "group6_d64": W.scaled(W.CONFIGS["tiny"], batch=2, num_q_heads=12, num_kv_heads=2, prefix=(0, 500), tree=(10, 50), max_depth=6),
    # odd number of KV heads: heads 0 and 1 share twin super-units, head 2's odd tile is split in halves between two CTAs
    "odd_heads_one_tile": W.scaled(W.CONFIGS["7b_mha"], batch=4, num_q_heads=12, num_kv_heads=3, prefix=(300, 2500), tree=(5, 30), max_depth=8),
    # one KV head, three query tiles: a pair plus a lone tile per sequence
    "single_head_three_tiles": W.scaled(W.CONFIGS["70b_gqa"], batch=3, num_q_heads=8, num_kv_heads=1, prefix=(100, 1800), tree=(36, 48)),
    # five KV heads, three query tiles each: pairs, twins and one lone tile in the same sequence
    "five_heads_three_tiles": W.scaled(W.CONFIGS["70b_gqa"], batch=2, num_q_heads=40, num_kv_heads=5, prefix=(400, 1500), tree=(40, 48)),
    "big_group_full_tree": W.scaled(W.CONFIGS["70b_gqa"], batch=2, num_q_heads=32, num_kv_heads=2, prefix=(130, 400),
                                    tree=(64, 64), max_depth=64, child_cap=0),
}


@pytest.mark.parametrize("name", list(CASES))
def test_attention_matches_oracle(E, oracle, name):
    cfg = CASES[name]
    inp = W.make_attn_inputs(cfg, capacity_pad=37)
    ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    out, status = _run(E, inp)
    assert status == 0
    _check(out, ref, inp.tree_sizes)


@pytest.mark.parametrize("splits", [1, 2, 3, 7, 64])
def test_forced_splits_agree(E, oracle, splits):
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=3, prefix=(60, 900), tree=(5, 40))
    inp = W.make_attn_inputs(cfg, salt=2)
    ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    out, status = _run(E, inp, num_splits=splits)
    assert status == 0
    _check(out, ref, inp.tree_sizes)
    again, _ = _run(E, inp, num_splits=splits)
    assert torch.equal(out.view(torch.int16), again.view(torch.int16)), "same call twice must be bit-identical"


def test_chain_tree_no_sizes_custom_scale(E, oracle):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=2, prefix=(0, 90), tree=(9, 9))
    inp = W.make_attn_inputs(cfg, salt=4, poison=True)
    inp.tree_parent[:] = torch.arange(-1, 8, dtype=torch.int32)
    assert int(inp.seq_lens.min()) >= 0
    ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, None, sm_scale=0.21)
    out, status = _run(E, inp, use_sizes=False, sm_scale=0.21)
    assert status == 0
    _check(out, ref, [9, 9])


@pytest.mark.parametrize("shape", ["ramp_up", "ramp_down", "late_spike"])
def test_reference_maximum_moves_between_steps(E, oracle, shape):
    """Scores that grow (or fall) by far more than the lazy-rescale threshold from one KV tile to the next: the shared
    reference maximum moves at many steps, the accumulator is rescaled, and the row sums of the softmax groups are
    handed over relative to different references.  Several query tiles, cut pieces and direct tiles are all present."""
    cfg = W.scaled(W.CONFIGS["70b_gqa"], batch=3, prefix=(700, 2600), tree=(20, 64))
    inp = W.make_attn_inputs(cfg, salt=11)
    S = inp.k_cache.shape[2]
    pos = torch.arange(S, dtype=torch.float32)
    if shape == "ramp_up":
        gain = 0.4 + pos / 128.0 * 0.35          # |q.k| grows by about 45 per tile: about 6 log2 units per tile after scaling
    elif shape == "ramp_down":
        gain = 0.4 + (S - pos) / 128.0 * 0.35
    else:
        gain = torch.where((pos > 900) & (pos < 1030), torch.tensor(6.0), torch.tensor(0.5))
    g = torch.Generator().manual_seed(21)
    # keys share a direction with the queries so that the dot products follow the gain instead of averaging out
    base = torch.randn(cfg.head_dim, generator=g).sign()
    k = (base[None, None, None, :] * gain[None, None, :, None] + 0.3 * torch.randn(inp.k_cache.shape, generator=g))
    inp.k_cache = k.to(torch.bfloat16)
    inp.q = (base[None, None, None, :] * 0.9 + 0.3 * torch.randn(inp.q.shape, generator=g)).to(torch.bfloat16)
    ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    for splits in (0, 3):
        out, status = _run(E, inp, num_splits=splits)
        assert status == 0
        _check(out, ref, inp.tree_sizes)


def _random_cfg(rng, i):
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 4, 5, 8]))
    G = int(rng.choice([1, 2, 3, 4, 8, 16]))
    lo = int(rng.choice([0, 0, 1, 100, 127, 128, 129, 600]))
    hi = lo + int(rng.choice([0, 1, 130, 700, 2500]))
    t_lo = int(rng.integers(0, 40))
    t_hi = int(rng.integers(max(t_lo, 1), 65))
    depth = int(rng.choice([2, 5, 9, 64]))
    shape = dict(max_depth=depth, child_cap=int(rng.choice([0, 2, 4])) if depth >= 9 else 0)   # (a capped shallow tree cannot hold 64 nodes)
    return W.scaled(W.CONFIGS["tiny"], batch=int(rng.integers(1, 7)), num_q_heads=Hkv * G, num_kv_heads=Hkv, head_dim=D,
                    prefix=(lo, hi), tree=(t_lo, t_hi), **shape)


@pytest.mark.parametrize("seed", range(int(os.environ.get("EAGLE_RANDOM_SHAPES", "24"))))
def test_random_shapes(E, oracle, seed):
    """Random head counts, group sizes, head dims, prefix ranges around the tile size and tree shapes, with the default
    split and with a forced one: every combination of pair / twin / lone super-units, one to many steps per item, empty
    trees and prefixes."""
    rng = np.random.default_rng(1000 + seed)
    cfg = _random_cfg(rng, seed)
    inp = W.make_attn_inputs(cfg, salt=seed, capacity_pad=int(rng.integers(0, 40)))
    ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    for splits in (0, int(rng.choice([2, 3, 5]))):
        out, status = _run(E, inp, num_splits=splits)
        assert status == 0, (cfg, splits)
        _check(out, ref, inp.tree_sizes)
        # the same keys and values behind a block table, in pages of a random size: same plan, same bits
        ps = int(rng.choice([16, 32, 64, 128, 256]))
        pk = W.make_paged_cache(inp, ps, salt=seed)
        d = torch.device("cuda:0")
        st = torch.zeros(1, dtype=torch.int32, device=d)
        paged = torch.full_like(out, float("nan")).to(d)
        E.eagle_tree_verify_attn_paged(inp.q.to(d), pk.k_pages.to(d), pk.v_pages.to(d), pk.block_table.to(d), inp.seq_lens.to(d),
                                       inp.tree_parent.to(d), paged, tree_sizes=inp.tree_sizes.to(d), num_splits=splits, status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0, (cfg, splits, ps)
        assert torch.equal(paged.cpu().view(torch.int16), out.view(torch.int16)), (cfg, splits, ps)


@pytest.mark.parametrize("seed", range(int(os.environ.get("EAGLE_RANDOM_BATCHES", "2"))))
def test_random_medium_batches(E, oracle, seed):
    """Batches large enough that every CTA team gets several items and most share boundaries cut a super-unit."""
    rng = np.random.default_rng(5000 + seed)
    Hkv, G = int(rng.choice([4, 8])), int(rng.choice([2, 4, 8]))
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=int(rng.integers(12, 28)), num_q_heads=Hkv * G, num_kv_heads=Hkv,
                   prefix=(int(rng.integers(0, 300)), int(rng.integers(1500, 5000))), tree=(int(rng.integers(1, 20)), 64))
    inp = W.make_attn_inputs(cfg, salt=100 + seed)
    ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    out, status = _run(E, inp)
    assert status == 0
    _check(out, ref, inp.tree_sizes)
    again, _ = _run(E, inp)
    assert torch.equal(out.view(torch.int16), again.view(torch.int16)), "same call twice must be bit-identical"


def test_empty_prefix_empty_tree_and_single_node(E, oracle):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=4, prefix=(0, 0), tree=(1, 6))
    inp = W.make_attn_inputs(cfg, salt=5)
    inp.tree_sizes[1] = 0
    inp.tree_sizes[2] = 1
    inp.seq_lens[3] = 70
    # regenerate the cache of sequence 3 so that its longer prefix is filled
    g = torch.Generator().manual_seed(5)
    cap = 70 + cfg.max_tree
    k = torch.full((4, cfg.num_kv_heads, cap, cfg.head_dim), float("nan"), dtype=torch.bfloat16)
    v = k.clone()
    k[:, :, :inp.kv_capacity] = inp.k_cache
    v[:, :, :inp.kv_capacity] = inp.v_cache
    k[3] = torch.randn(k[3].shape, generator=g).to(torch.bfloat16)
    v[3] = torch.randn(v[3].shape, generator=g).to(torch.bfloat16)
    inp.k_cache, inp.v_cache = k, v
    ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    out, status = _run(E, inp)
    assert status == 0
    _check(out, ref, inp.tree_sizes)


def test_invalid_inputs_are_reported_not_trapped(E, oracle):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=3, prefix=(20, 50), tree=(4, 8))
    inp = W.make_attn_inputs(cfg, salt=6)
    good_ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    bad = W.make_attn_inputs(cfg, salt=6)
    bad.tree_parent[1, 2] = 2          # parent must be < node index
    out, status = _run(E, bad)
    assert status == -5
    got = out.double().numpy()
    assert np.all(got[1] == 0.0)       # the invalid sequence is zeroed
    for b in (0, 2):                   # the others are still right
        n = int(inp.tree_sizes[b])
        assert np.abs(got[b, :n] - good_ref[b, :n]).max() <= MAX_ABS
    bad2 = W.make_attn_inputs(cfg, salt=6)
    bad2.seq_lens[0] = bad2.kv_capacity   # prefix + tree does not fit the cache
    out, status = _run(E, bad2)
    assert status == -6 and np.all(out.double().numpy()[0] == 0.0)


def test_piece_in_which_a_row_sees_no_key(E, oracle):
    """Prefix of 100 slots and a star tree of 64 nodes (every node sees the prefix and itself only), cut into two pieces
    at the KV-tile boundary: in the second piece (tree nodes 28..63) the rows of nodes 0..27 have every key masked, so
    their partial must not count in the merge.  Also with a chain, where the late rows see everything."""
    cfg = W.scaled(W.CONFIGS["tiny"], batch=3, num_q_heads=8, num_kv_heads=2, head_dim=128, prefix=(100, 100), tree=(64, 64), max_depth=64)
    for shape in ("star", "chain"):
        inp = W.make_attn_inputs(cfg, salt=31)
        inp.tree_parent[:] = -1 if shape == "star" else torch.arange(-1, 63, dtype=torch.int32)
        ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
        for splits in (2, 0):
            out, status = _run(E, inp, num_splits=splits)
            assert status == 0
            _check(out, ref, inp.tree_sizes)


def test_plan_once_attend_many_layers(E, oracle):
    """One plan for a verification pass, then attention + combine per layer on that plan: bit for bit what the one-call
    form gives for every layer's K/V, and the oracle's result; the plan's own tree masks equal the oracle's bit for bit."""
    d = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=9, prefix=(30, 2500), tree=(0, 64), max_depth=64)
    layers = [W.make_attn_inputs(cfg, salt=40)]
    for l in (1, 2):
        other = W.make_attn_inputs(cfg, salt=40)
        g = torch.Generator().manual_seed(400 + l)
        for name in ("q", "k_cache", "v_cache"):
            t = getattr(other, name)
            fresh = torch.randn(t.shape, generator=g).to(torch.bfloat16)
            setattr(other, name, torch.where(torch.isnan(t), t, fresh))     # same lengths and trees, other values
        layers.append(other)
    base = layers[0]
    status = torch.zeros(1, dtype=torch.int32, device=d)
    for splits in (0, 3):
        plan = E.eagle_tree_verify_plan(tuple(base.q.shape), cfg.num_kv_heads, base.k_cache.shape[2], base.seq_lens.to(d),
                                        base.tree_parent.to(d), tree_sizes=base.tree_sizes.to(d), num_splits=splits, status=status)
        torch.cuda.synchronize()
        anc_ref, _ = oracle.tree_ancestors(base.tree_parent.numpy(), base.tree_sizes.numpy())
        assert np.array_equal(plan.masks().cpu().numpy().view(np.uint64), anc_ref)
        for inp in layers:
            out = torch.full(inp.q.shape, float("nan"), dtype=torch.bfloat16, device=d)
            plan.attend(inp.q.to(d), inp.k_cache.to(d), inp.v_cache.to(d), out, status=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            whole, st = _run(E, inp, num_splits=splits)
            assert st == 0 and torch.equal(out.cpu().view(torch.int16), whole.view(torch.int16))
            ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
            _check(out.cpu(), ref, inp.tree_sizes)
    # the same over a paged cache
    pk = W.make_paged_cache(base, 64, salt=3)
    plan = E.eagle_tree_verify_plan(tuple(base.q.shape), cfg.num_kv_heads, 0, base.seq_lens.to(d), base.tree_parent.to(d),
                                    tree_sizes=base.tree_sizes.to(d), status=status,
                                    paged=(pk.block_table.to(d), pk.k_pages.shape[0], pk.page_size))
    out = plan.attend_paged(base.q.to(d), pk.k_pages.to(d), pk.v_pages.to(d), pk.block_table.to(d), status=status)
    torch.cuda.synchronize()
    whole, st = _run(E, base)
    assert int(status.item()) == 0 and torch.equal(out.cpu().view(torch.int16), whole.view(torch.int16))


def test_planner_masks_match_oracle(E, oracle):
    """The masks the attention kernel really reads (built by the planner, left in the workspace), bit for bit; trees of
    every size up to 64 and depth up to 64, per sequence and one tree shared by all."""
    d = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=70, num_q_heads=8, num_kv_heads=2, prefix=(0, 300), tree=(0, 64), max_depth=64)
    sizes, parent = W.make_trees(cfg, salt=8)
    lens = torch.randint(0, 300, (cfg.batch,), dtype=torch.int32)
    anc_ref, _ = oracle.tree_ancestors(parent.numpy(), sizes.numpy())
    status = torch.zeros(1, dtype=torch.int32, device=d)
    plan = E.eagle_tree_verify_plan((cfg.batch, 64, 8, 128), 2, 400, lens.to(d), parent.to(d), tree_sizes=sizes.to(d), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(plan.masks().cpu().numpy().view(np.uint64), anc_ref)
    b = int(sizes.argmax())
    plan = E.eagle_tree_verify_plan((cfg.batch, 64, 8, 128), 2, 400, lens.to(d), parent[b].contiguous().to(d),
                                    tree_sizes=sizes[b:b + 1].to(d), status=status, shared_tree=True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(plan.masks().cpu().numpy().view(np.uint64), np.broadcast_to(anc_ref[b], anc_ref.shape))


def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_fine(E, oracle):
    """Failure handling: every wait in the attention kernel is bounded.  The K/V producer is told (test hook) to fall
    silent after two tiles and the limit is lowered to 2 ms: the kernel must return by itself with EAGLE_ERR_TIMEOUT,
    and an ordinary call right after must be correct."""
    d = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["tiny"], batch=2, prefix=(600, 900))
    inp = W.make_attn_inputs(cfg, salt=12)
    ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    try:
        E.set_wait_limit_ns(2_000_000)
        E.test_stall_kv_producer(2)
        out, status = _run(E, inp)
    finally:
        E.test_stall_kv_producer(-1)
        E.set_wait_limit_ns(0)
    assert status == -8, E.status_string(status)
    out, status = _run(E, inp)
    assert status == 0
    _check(out, ref, inp.tree_sizes)


def test_mask_builder_matches_oracle(E, oracle):
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=50, tree=(0, 64), max_depth=64)
    sizes, parent = W.make_trees(cfg, salt=7)
    anc_ref, depth_ref = oracle.tree_ancestors(parent.numpy(), sizes.numpy())
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    anc, depth = E.eagle_tree_build_mask(parent.cuda(), sizes.cuda(), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(anc.cpu().numpy().view(np.uint64), anc_ref)
    assert np.array_equal(depth.cpu().numpy().astype(np.int32), depth_ref)


@pytest.mark.parametrize("name", ["mixtral_gqa", "serving_mix"])
def test_full_size_sampled_rows(E, oracle, name):
    """Full BASELINE sizes in the bench's launch configuration; the oracle checks sampled (sequence, KV head)
    units, and cheap properties are checked everywhere."""
    cfg = W.CONFIGS[name]
    inp = W.make_attn_inputs(cfg)
    out, status = _run(E, inp)
    assert status == 0
    got = out.double().numpy()
    assert np.isfinite(got).all()
    for b in range(cfg.batch):
        assert np.all(got[b, int(inp.tree_sizes[b]):] == 0.0)
    G = cfg.num_q_heads // cfg.num_kv_heads
    rng = np.random.default_rng(0)
    lens = inp.seq_lens.numpy()
    picks = {(int(np.argmax(lens)), 0), (int(np.argmin(lens)), cfg.num_kv_heads - 1)}
    while len(picks) < 4:
        picks.add((int(rng.integers(cfg.batch)), int(rng.integers(cfg.num_kv_heads))))
    for b, g in sorted(picks):
        n = int(inp.tree_sizes[b])
        end = int(lens[b]) + n
        ref = oracle.tree_verify_attn(inp.q[b:b + 1, :, g * G:(g + 1) * G].contiguous(),
                                      inp.k_cache[b:b + 1, g:g + 1, :end].contiguous(),
                                      inp.v_cache[b:b + 1, g:g + 1, :end].contiguous(),
                                      inp.seq_lens[b:b + 1], inp.tree_parent[b:b + 1], inp.tree_sizes[b:b + 1])
        err = np.abs(got[b, :n, g * G:(g + 1) * G] - ref[0, :n])
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (b, g, err.max(), err.mean())
