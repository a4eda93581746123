"""Parity of the tree attention over an fp8 (e4m3) cache (through the C ABI) with the oracle's fp8 form.  Needs a B200.

Only the storage differs from the bf16 call: the codes are widened exactly, the scales are applied in fp32, so the same
bounds hold against the oracle evaluated on the same codes and scales."""
import os

import numpy as np
import pytest
import torch

from paper_2401_15077_b200 import workloads as W

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 2e-2, 2e-3


@pytest.fixture(scope="module")
def E():
    from paper_2401_15077_b200 import build, binding
    build.build()
    binding.load()
    assert torch.cuda.is_available()
    return binding


def _run(E, inp, f8, num_splits=0, sm_scale=0.0):
    d = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=d)
    out = torch.full(inp.q.shape, float("nan"), dtype=torch.bfloat16, device=d)
    E.eagle_tree_verify_attn_fp8(inp.q.to(d), f8.k_codes.to(d), f8.v_codes.to(d), f8.k_scale.to(d), f8.v_scale.to(d), inp.seq_lens.to(d),
                                 inp.tree_parent.to(d), out, tree_sizes=inp.tree_sizes.to(d), num_splits=num_splits, status=status,
                                 sm_scale=sm_scale)
    torch.cuda.synchronize()
    return out.cpu(), int(status.item())


def _check(out, ref, sizes, scale=1.0):
    got = out.double().numpy()
    assert np.isfinite(got).all()
    rows = np.zeros(ref.shape[:2], bool)
    for b, n in enumerate(sizes):
        rows[b, :int(n)] = True
        assert np.all(got[b, int(n):] == 0.0)
    if rows.any():
        err = np.abs(got - ref)[rows]
        assert err.max() <= MAX_ABS * scale and err.mean() <= MEAN_ABS * scale, (err.max(), err.mean())


CASES = {
    "7b_mha": W.CONFIGS["7b_mha"],
    "70b_gqa_b2": W.scaled(W.CONFIGS["70b_gqa"], batch=2),
    "mixtral_gqa_small": W.scaled(W.CONFIGS["mixtral_gqa"], batch=2, prefix=(1500, 3000)),
    "serving_mix_small": W.scaled(W.CONFIGS["serving_mix"], batch=6, prefix=(100, 1500)),
    "ragged_small_trees": W.scaled(W.CONFIGS["7b_mha"], batch=5, num_q_heads=16, num_kv_heads=4, prefix=(0, 700), tree=(0, 33)),
    "group3": W.scaled(W.CONFIGS["7b_mha"], batch=3, num_q_heads=12, num_kv_heads=4, prefix=(50, 1200), tree=(3, 64), max_depth=8),
    "odd_heads": W.scaled(W.CONFIGS["7b_mha"], batch=4, num_q_heads=12, num_kv_heads=3, prefix=(300, 2500), tree=(5, 30), max_depth=8),
    "five_heads_three_tiles": W.scaled(W.CONFIGS["70b_gqa"], batch=2, num_q_heads=40, num_kv_heads=5, prefix=(400, 1500), tree=(40, 48)),
}


@pytest.mark.parametrize("name", list(CASES))
def test_fp8_attention_matches_oracle(E, oracle, name):
    cfg = CASES[name]
    inp = W.make_attn_inputs(cfg, salt=3, capacity_pad=19)
    f8 = W.make_fp8_cache(inp)
    ref = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, f8.v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    for splits in (0, 3):
        out, status = _run(E, inp, f8, num_splits=splits)
        assert status == 0
        _check(out, ref, inp.tree_sizes)
    again, _ = _run(E, inp, f8, num_splits=3)
    assert torch.equal(out.view(torch.int16), again.view(torch.int16))


@pytest.mark.parametrize("seed", range(int(os.environ.get("EAGLE_RANDOM_FP8", "8"))))
def test_random_shapes_fp8(E, oracle, seed):
    """Random head counts, group sizes (those that divide 128 and those that do not: the two ways a query tile is staged),
    prefix ranges around the tile size and tree shapes, default split and a forced one, twice each (bit-identical)."""
    rng = np.random.default_rng(7000 + seed)
    Hkv = int(rng.choice([1, 2, 3, 5, 8]))
    G = int(rng.choice([1, 2, 3, 4, 6, 8, 16]))
    lo = int(rng.choice([0, 0, 1, 100, 127, 128, 129, 600]))
    hi = lo + int(rng.choice([0, 1, 130, 700, 2500]))
    t_lo = int(rng.integers(0, 40))
    t_hi = int(rng.integers(max(t_lo, 1), 65))
    depth = int(rng.choice([2, 5, 9, 64]))
    shape = dict(max_depth=depth, child_cap=int(rng.choice([0, 2, 4])) if depth >= 9 else 0)
    cfg = W.scaled(W.CONFIGS["7b_mha"], batch=int(rng.integers(1, 7)), num_q_heads=Hkv * G, num_kv_heads=Hkv, prefix=(lo, hi),
                   tree=(t_lo, t_hi), **shape)
    inp = W.make_attn_inputs(cfg, salt=seed, capacity_pad=int(rng.integers(0, 40)))
    f8 = W.make_fp8_cache(inp)
    ref = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, f8.v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    for splits in (0, int(rng.choice([2, 3, 5]))):
        out, status = _run(E, inp, f8, num_splits=splits)
        assert status == 0, (cfg, splits)
        _check(out, ref, inp.tree_sizes)
        again, _ = _run(E, inp, f8, num_splits=splits)
        assert torch.equal(out.view(torch.int16), again.view(torch.int16)), (cfg, splits)


def test_every_code_is_widened_exactly(E, oracle):
    """Keys of zeros (uniform softmax) and values that run through all 254 number codes, subnormals included: the output
    is the mean of the decoded values, so a wrongly widened code shows.  Large and small scales per head."""
    cfg = W.scaled(W.CONFIGS["7b_mha"], batch=2, num_q_heads=4, num_kv_heads=2, prefix=(508, 508), tree=(4, 4))
    inp = W.make_attn_inputs(cfg, salt=1)
    S = inp.k_cache.shape[2]
    codes = torch.tensor([c for c in range(256) if c not in (0x7F, 0xFF)], dtype=torch.uint8)
    g = torch.Generator().manual_seed(9)
    v_codes = codes[torch.randint(0, 254, (2, 2, S, 128), generator=g)]
    # column d of slot j holds a code that depends on (j + d): every column's mean runs over all codes
    k_codes = torch.zeros((2, 2, S, 128), dtype=torch.uint8)
    k_scale = torch.ones((2, 2))
    v_scale = torch.tensor([[1.0, 2.0 ** -7], [3.0, 0.011]])
    f8 = W.Fp8KV(k_codes, v_codes, k_scale, v_scale)
    ref = oracle.tree_verify_attn_fp8(inp.q, k_codes, v_codes, k_scale, v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    out, status = _run(E, inp, f8)
    assert status == 0
    got = out.double().numpy()
    for b in range(2):
        for h in range(4):
            s = float(v_scale[b, h // 2])
            err = np.abs(got[b, :4, h] - ref[b, :4, h])
            assert err.max() <= 2e-2 * s * 16, (b, h, err.max())         # values up to 448 * scale: bf16 rounding of means ~ 10 * scale
            assert err.max() <= np.abs(ref[b, :4, h]).max() * 2.0 ** -7 + 1e-6 * s
    # only subnormal codes (|value| <= 7 * 2^-9): a flush to zero in the widening would return zeros
    sub = torch.tensor([1, 2, 3, 4, 5, 6, 7], dtype=torch.uint8)
    v_sub = sub[torch.randint(0, 7, (2, 2, S, 128), generator=g)]
    f8s = W.Fp8KV(k_codes, v_sub, k_scale, torch.full((2, 2), 64.0))
    ref = oracle.tree_verify_attn_fp8(inp.q, k_codes, v_sub, k_scale, f8s.v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    out, status = _run(E, inp, f8s)
    got = out.double().numpy()[:, :4]
    assert status == 0 and ref[:, :4].min() > 0.3 and np.abs(got - ref[:, :4]).max() <= 2e-2


def test_fp8_plan_once_attend_many(E, oracle):
    d = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=7, prefix=(30, 2000), tree=(0, 64), max_depth=64)
    inp = W.make_attn_inputs(cfg, salt=5)
    f8 = W.make_fp8_cache(inp)
    status = torch.zeros(1, dtype=torch.int32, device=d)
    plan = E.eagle_tree_verify_plan(tuple(inp.q.shape), cfg.num_kv_heads, inp.k_cache.shape[2], inp.seq_lens.to(d), inp.tree_parent.to(d),
                                    tree_sizes=inp.tree_sizes.to(d), status=status)
    out = plan.attend_fp8(inp.q.to(d), f8.k_codes.to(d), f8.v_codes.to(d), f8.k_scale.to(d), f8.v_scale.to(d), status=status)
    torch.cuda.synchronize()
    whole, st = _run(E, inp, f8)
    assert st == 0 and int(status.item()) == 0 and torch.equal(out.cpu().view(torch.int16), whole.view(torch.int16))
    ref = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, f8.v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    _check(whole, ref, inp.tree_sizes)


def test_fp8_full_size_mixtral_sampled(E, oracle):
    cfg = W.CONFIGS["mixtral_gqa"]
    inp = W.make_attn_inputs(cfg)
    f8 = W.make_fp8_cache(inp)
    out, status = _run(E, inp, f8)
    assert status == 0
    got = out.double().numpy()
    assert np.isfinite(got).all()
    G = cfg.num_q_heads // cfg.num_kv_heads
    for b, g in [(0, 0), (7, 7), (3, 5)]:
        n, end = int(inp.tree_sizes[b]), int(inp.seq_lens[b] + inp.tree_sizes[b])
        ref = oracle.tree_verify_attn_fp8(inp.q[b:b + 1, :, g * G:(g + 1) * G].contiguous(), f8.k_codes[b:b + 1, g:g + 1, :end].contiguous(),
                                          f8.v_codes[b:b + 1, g:g + 1, :end].contiguous(), f8.k_scale[b:b + 1, g:g + 1].contiguous(),
                                          f8.v_scale[b:b + 1, g:g + 1].contiguous(), inp.seq_lens[b:b + 1], inp.tree_parent[b:b + 1],
                                          inp.tree_sizes[b:b + 1])
        err = np.abs(got[b, :n, g * G:(g + 1) * G] - ref[0, :n])
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (b, g, err.max(), err.mean())


def test_fp8_refuses_unsupported_shapes(E):
    d = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["tiny"], batch=1)                     # head_dim 64
    inp = W.make_attn_inputs(cfg)
    f8 = W.make_fp8_cache(inp)
    with pytest.raises(E.EagleError):
        E.eagle_tree_verify_attn_fp8(inp.q.to(d), f8.k_codes.to(d), f8.v_codes.to(d), f8.k_scale.to(d), f8.v_scale.to(d),
                                     inp.seq_lens.to(d), inp.tree_parent.to(d))


def test_fp8_many_short_items_repeatedly(E, oracle):
    """A small ragged batch gives every CTA items of one or two KV tiles; the last tile of a sequence (whose V rows past
    prefix + tree are zeroed in shared memory) then shares its ring slot with a tile that may not have been consumed yet.
    The call is repeated: every run must be within the bounds and bit-identical to the first (a race here showed as a
    wrong (sequence, KV head) unit in about half of the runs)."""
    cfg = CASES["ragged_small_trees"]
    inp = W.make_attn_inputs(cfg, salt=3, capacity_pad=19)
    f8 = W.make_fp8_cache(inp)
    ref = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, f8.v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    first = None
    for rep in range(30):
        out, status = _run(E, inp, f8)
        assert status == 0
        _check(out, ref, inp.tree_sizes)
        if first is None:
            first = out
        assert torch.equal(out.view(torch.int16), first.view(torch.int16)), rep


def test_fp8_wait_that_runs_out_is_reported(E, oracle):
    """The converter warps' waits are bounded like every other: with the K/V producer silenced after two tiles (test hook)
    and the limit lowered to 2 ms the call returns by itself with EAGLE_ERR_TIMEOUT; the next call is correct."""
    cfg = W.scaled(W.CONFIGS["7b_mha"], batch=2, num_q_heads=8, num_kv_heads=2, prefix=(600, 900), tree=(8, 8))
    inp = W.make_attn_inputs(cfg, salt=12)
    f8 = W.make_fp8_cache(inp)
    ref = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, f8.v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    try:
        E.set_wait_limit_ns(2_000_000)
        E.test_stall_kv_producer(2)
        out, status = _run(E, inp, f8)
    finally:
        E.test_stall_kv_producer(-1)
        E.set_wait_limit_ns(0)
    assert status == -8, E.status_string(status)
    out, status = _run(E, inp, f8)
    assert status == 0
    _check(out, ref, inp.tree_sizes)


# ---- the fp8 cache kept in pages

def _run_paged(E, inp, f8, pk, num_splits=0):
    d = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=d)
    out = torch.full(inp.q.shape, float("nan"), dtype=torch.bfloat16, device=d)
    E.eagle_tree_verify_attn_paged_fp8(inp.q.to(d), pk.k_pages.to(d), pk.v_pages.to(d), f8.k_scale.to(d), f8.v_scale.to(d),
                                       pk.block_table.to(d), inp.seq_lens.to(d), inp.tree_parent.to(d), out,
                                       tree_sizes=inp.tree_sizes.to(d), num_splits=num_splits, status=status)
    torch.cuda.synchronize()
    return out.cpu(), int(status.item())


@pytest.mark.parametrize("page_size", [16, 64, 128, 256])
@pytest.mark.parametrize("name", ["serving_mix_small", "ragged_small_trees", "group3", "five_heads_three_tiles"])
def test_paged_fp8_matches_oracle_and_the_contiguous_call(E, oracle, name, page_size):
    """Pages of codes behind a block table (pages scattered over the pool, unused rows and spare pages hold the NaN code):
    the oracle's paged fp8 form within the bounds, and the contiguous fp8 call bit for bit (same plan, same arithmetic)."""
    cfg = CASES[name]
    inp = W.make_attn_inputs(cfg, salt=11, capacity_pad=19)
    f8 = W.make_fp8_cache(inp)
    pk = W.make_paged_cache(inp, page_size, salt=page_size, codes=f8)
    ref = oracle.tree_verify_attn_fp8_paged(inp.q, pk.k_pages, pk.v_pages, f8.k_scale, f8.v_scale, pk.block_table, inp.seq_lens,
                                            inp.tree_parent, inp.tree_sizes)
    for splits in (0, 3):
        out, status = _run_paged(E, inp, f8, pk, num_splits=splits)
        assert status == 0, (name, page_size, splits)
        _check(out, ref, inp.tree_sizes)
        flat, st = _run(E, inp, f8, num_splits=splits)
        assert st == 0 and torch.equal(out.view(torch.int16), flat.view(torch.int16)), (name, page_size, splits)


def test_paged_fp8_plan_once_attend_many_and_bad_page(E, oracle):
    d = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=6, prefix=(30, 1500), tree=(0, 64), max_depth=64)
    inp = W.make_attn_inputs(cfg, salt=6)
    f8 = W.make_fp8_cache(inp)
    pk = W.make_paged_cache(inp, 32, salt=2, codes=f8)
    status = torch.zeros(1, dtype=torch.int32, device=d)
    plan = E.eagle_tree_verify_plan(tuple(inp.q.shape), cfg.num_kv_heads, 0, inp.seq_lens.to(d), inp.tree_parent.to(d),
                                    tree_sizes=inp.tree_sizes.to(d), status=status,
                                    paged=(pk.block_table.to(d), pk.k_pages.shape[0], pk.page_size))
    out = plan.attend_paged_fp8(inp.q.to(d), pk.k_pages.to(d), pk.v_pages.to(d), f8.k_scale.to(d), f8.v_scale.to(d),
                                pk.block_table.to(d), status=status)
    torch.cuda.synchronize()
    whole, st = _run_paged(E, inp, f8, pk)
    assert st == 0 and int(status.item()) == 0 and torch.equal(out.cpu().view(torch.int16), whole.view(torch.int16))
    ref = oracle.tree_verify_attn_fp8_paged(inp.q, pk.k_pages, pk.v_pages, f8.k_scale, f8.v_scale, pk.block_table, inp.seq_lens,
                                            inp.tree_parent, inp.tree_sizes)
    _check(whole, ref, inp.tree_sizes)
    # a visible slot whose page is outside the pool: that sequence is refused and zeroed, the others are untouched
    b = int(torch.nonzero(inp.tree_sizes > 0)[0])
    bad = W.PagedKV(pk.k_pages, pk.v_pages, pk.block_table.clone(), pk.page_size)
    bad.block_table[b, 0] = pk.k_pages.shape[0]
    got, st = _run_paged(E, inp, f8, bad)
    assert st == -11          # EAGLE_ERR_PAGE
    assert torch.all(got[b] == 0)
    sizes = inp.tree_sizes.clone()       # (the work is split differently without that sequence: the others agree with
    sizes[b] = 0                         # the oracle within the bounds, not with the first call bit for bit)
    ref[b] = 0.0
    _check(got, ref, sizes)
