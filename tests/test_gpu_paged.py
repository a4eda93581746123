"""Parity of the CUDA tree attention over a paged cache, and with one tree shared by every sequence, with the fp64
oracle.  Needs a B200."""
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


def _run_paged(E, inp, pk, **kw):
    d = torch.device("cuda:0")
    q = inp.q.to(d)
    out = torch.full_like(q, float("nan"))
    status = torch.zeros(1, dtype=torch.int32, device=d)
    E.eagle_tree_verify_attn_paged(q, pk.k_pages.to(d), pk.v_pages.to(d), pk.block_table.to(d), inp.seq_lens.to(d),
                                   inp.tree_parent.to(d), out, tree_sizes=inp.tree_sizes.to(d), status=status, **kw)
    torch.cuda.synchronize()
    return out.cpu(), int(status.item())


CASES = {
    "tiny": W.CONFIGS["tiny"],
    "d64_gqa_ragged": W.scaled(W.CONFIGS["tiny"], batch=5, num_q_heads=16, num_kv_heads=4, prefix=(0, 700), tree=(1, 33)),
    "serving_mix_small": W.scaled(W.CONFIGS["serving_mix"], batch=6, prefix=(100, 1500)),
    "odd_heads_one_tile": W.scaled(W.CONFIGS["7b_mha"], batch=4, num_q_heads=12, num_kv_heads=3, prefix=(300, 2500), tree=(5, 30),
                                   max_depth=8),
    "70b_gqa_b2": W.scaled(W.CONFIGS["70b_gqa"], batch=2),
}


@pytest.mark.parametrize("page_size", [16, 32, 64, 128, 256])
@pytest.mark.parametrize("name", list(CASES))
def test_paged_attention_matches_oracle(E, oracle, name, page_size):
    cfg = CASES[name]
    inp = W.make_attn_inputs(cfg, capacity_pad=37)
    pk = W.make_paged_cache(inp, page_size, salt=page_size)
    ref = oracle.tree_verify_attn_paged(inp.q, pk.k_pages, pk.v_pages, pk.block_table, inp.seq_lens, inp.tree_parent,
                                        inp.tree_sizes)
    out, status = _run_paged(E, inp, pk)
    assert status == 0
    _check(out, ref, inp.tree_sizes)


def test_paged_equals_contiguous_bitwise(E):
    """Same keys, same plan, same arithmetic: the two cache layouts give identical bits."""
    cfg = CASES["serving_mix_small"]
    inp = W.make_attn_inputs(cfg)
    d = torch.device("cuda:0")
    q = inp.q.to(d)
    a = E.eagle_tree_verify_attn(q, inp.k_cache.to(d), inp.v_cache.to(d), inp.seq_lens.to(d), inp.tree_parent.to(d),
                                 tree_sizes=inp.tree_sizes.to(d))
    for ps in (16, 128):
        pk = W.make_paged_cache(inp, ps, salt=7)
        b, status = _run_paged(E, inp, pk)
        assert status == 0
        assert torch.equal(a.cpu().view(torch.int16), b.view(torch.int16))


def test_paged_forced_splits(E, oracle):
    cfg = CASES["d64_gqa_ragged"]
    inp = W.make_attn_inputs(cfg)
    pk = W.make_paged_cache(inp, 32, salt=1)
    ref = oracle.tree_verify_attn_paged(inp.q, pk.k_pages, pk.v_pages, pk.block_table, inp.seq_lens, inp.tree_parent,
                                        inp.tree_sizes)
    out, status = _run_paged(E, inp, pk, num_splits=3)
    assert status == 0
    _check(out, ref, inp.tree_sizes)


def test_bad_page_is_reported_and_the_sequence_zeroed(E, oracle):
    cfg = CASES["d64_gqa_ragged"]
    inp = W.make_attn_inputs(cfg)
    pk = W.make_paged_cache(inp, 16, salt=2)
    ref = oracle.tree_verify_attn_paged(inp.q, pk.k_pages, pk.v_pages, pk.block_table, inp.seq_lens, inp.tree_parent,
                                        inp.tree_sizes)
    bad = 2
    used = (int(inp.seq_lens[bad]) + int(inp.tree_sizes[bad]) + 15) // 16
    pk.block_table[bad, used - 1] = pk.k_pages.shape[0]      # one past the pool
    out, status = _run_paged(E, inp, pk)
    assert status == -11
    got = out.double().numpy()
    assert np.all(got[bad] == 0.0)
    sizes = inp.tree_sizes.clone()
    sizes[bad] = 0
    ref[bad] = 0.0
    _check(out, ref, sizes)


def test_capacity_is_pages_times_page_size(E):
    cfg = CASES["tiny"]
    inp = W.make_attn_inputs(cfg)
    pk = W.make_paged_cache(inp, 64, salt=3)
    pk.block_table = pk.block_table[:, :4].contiguous()     # 256 slots: the prefix alone fills them, the tree does not fit
    out, status = _run_paged(E, inp, pk)
    assert status == -6
    assert torch.all(out == 0)


def test_paged_host_checks(E):
    cfg = CASES["tiny"]
    inp = W.make_attn_inputs(cfg)
    d = torch.device("cuda:0")
    q = inp.q.to(d)
    for ps in (8, 24):     # too small; not a power of two
        k = torch.zeros((4, cfg.num_kv_heads, ps, cfg.head_dim), dtype=torch.bfloat16, device=d)
        table = torch.zeros((cfg.batch, 64), dtype=torch.int32, device=d)
        with pytest.raises(E.EagleError):
            E.eagle_tree_verify_attn_paged(q, k, k, table, inp.seq_lens.to(d), inp.tree_parent.to(d))


# ---- one tree shared by every sequence

@pytest.mark.parametrize("name", ["d64_gqa_ragged", "70b_gqa_b2"])
def test_shared_tree_matches_oracle(E, oracle, name):
    cfg = CASES[name]
    inp = W.make_attn_inputs(cfg)
    B = cfg.batch
    n0 = int(inp.tree_sizes[0])
    # every sequence uses sequence 0's tree; keys and values of the tree sit at L_b + m, so rebuild the inputs with equal sizes
    sizes = torch.full((B,), n0, dtype=torch.int32)
    parent = inp.tree_parent[0:1].expand(B, -1).contiguous()
    lens = torch.minimum(inp.seq_lens, torch.tensor(inp.kv_capacity - n0, dtype=torch.int32)).clamp(min=0)
    k = torch.where(torch.isnan(inp.k_cache.float()), torch.zeros((), dtype=torch.float32), inp.k_cache.float()).to(torch.bfloat16)
    v = torch.where(torch.isnan(inp.v_cache.float()), torch.zeros((), dtype=torch.float32), inp.v_cache.float()).to(torch.bfloat16)
    qq = torch.where(torch.isnan(inp.q.float()), torch.zeros((), dtype=torch.float32), inp.q.float()).to(torch.bfloat16)
    ref = oracle.tree_verify_attn(qq, k, v, lens, parent, sizes)
    d = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=d)
    out = E.eagle_tree_verify_attn(qq.to(d), k.to(d), v.to(d), lens.to(d), inp.tree_parent[0].contiguous().to(d),
                                   tree_sizes=sizes[:1].to(d), status=status, shared_tree=True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    _check(out.cpu(), ref, sizes)
    # and identical bits to the call that is given the tree once per sequence
    per_seq = E.eagle_tree_verify_attn(qq.to(d), k.to(d), v.to(d), lens.to(d), parent.to(d), tree_sizes=sizes.to(d))
    assert torch.equal(out.view(torch.int16), per_seq.view(torch.int16))


# ---- commit of the accepted path on a paged cache (bit exact)

def _bits(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


COMMIT_CASES = {
    "tiny": W.CONFIGS["tiny"],
    "mix_small": W.scaled(W.CONFIGS["serving_mix"], batch=12, prefix=(0, 700)),
    "d64_deep_chains": W.scaled(W.CONFIGS["tiny"], batch=9, num_q_heads=6, num_kv_heads=3, prefix=(0, 90), tree=(40, 64), max_depth=64,
                                child_cap=2),
}


@pytest.mark.parametrize("page_size", [16, 64, 256])
@pytest.mark.parametrize("name", list(COMMIT_CASES))
def test_paged_commit_matches_oracle(E, oracle, name, page_size):
    cfg = COMMIT_CASES[name]
    d = torch.device("cuda:0")
    moved = 0
    for salt in range(2):
        inp = W.make_attn_inputs(cfg, salt=salt, poison=False, capacity_pad=5)
        pk = W.make_paged_cache(inp, page_size, salt=salt, poison=False)
        paths = W.make_accepted_paths(inp.tree_sizes, inp.tree_parent, cfg.max_tree, cfg.index, salt)
        g = torch.Generator().manual_seed(W.seed_for(cfg.index, "features", salt))
        feats = torch.randn((cfg.batch, cfg.max_tree, 64), generator=g).to(torch.bfloat16)
        ref = oracle.tree_commit_paged(pk.k_pages, pk.v_pages, pk.block_table, inp.seq_lens, paths, cfg.max_tree)
        ref_f = oracle.tree_commit(inp.k_cache, inp.v_cache, inp.seq_lens, paths, cfg.max_tree, features=feats)["features_out"]
        kd, vd = pk.k_pages.to(d), pk.v_pages.to(d)
        status = torch.zeros(1, dtype=torch.int32, device=d)
        new_len, fout = E.eagle_tree_commit_paged(kd, vd, pk.block_table.to(d), inp.seq_lens.to(d), paths.to(d), cfg.max_tree,
                                                  features=feats.to(d), status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and ref["valid"].all()
        assert np.array_equal(_bits(kd), ref["k_pages"]) and np.array_equal(_bits(vd), ref["v_pages"])
        assert np.array_equal(new_len.cpu().numpy(), ref["new_seq_lens"])
        assert np.array_equal(_bits(fout), ref_f)
        moved += int((ref["new_seq_lens"] - inp.seq_lens.numpy()).sum())
    assert moved > 0


def test_paged_commit_bad_page_and_bad_path(E, oracle):
    cfg = COMMIT_CASES["mix_small"]
    d = torch.device("cuda:0")
    inp = W.make_attn_inputs(cfg, poison=False)
    pk = W.make_paged_cache(inp, 16, poison=False)
    paths = W.make_accepted_paths(inp.tree_sizes, inp.tree_parent, cfg.max_tree, cfg.index)
    lens = [int((paths[b] >= 0).sum()) for b in range(cfg.batch)]
    victim = max(range(cfg.batch), key=lambda b: lens[b])
    assert lens[victim] >= 1
    L = int(inp.seq_lens[victim])
    pk.block_table[victim, (L + int(paths[victim, lens[victim] - 1])) // 16] = -5
    ref = oracle.tree_commit_paged(pk.k_pages, pk.v_pages, pk.block_table, inp.seq_lens, paths, cfg.max_tree)
    assert ref["valid"][victim] == 0
    kd, vd = pk.k_pages.to(d), pk.v_pages.to(d)
    status = torch.zeros(1, dtype=torch.int32, device=d)
    new_len, _ = E.eagle_tree_commit_paged(kd, vd, pk.block_table.to(d), inp.seq_lens.to(d), paths.to(d), cfg.max_tree, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == -11
    assert np.array_equal(_bits(kd), ref["k_pages"]) and np.array_equal(_bits(vd), ref["v_pages"])
    assert np.array_equal(new_len.cpu().numpy(), ref["new_seq_lens"])


def test_verify_then_commit_then_verify_on_pages(E, oracle):
    """The step as a serving loop runs it: attention over the pages, commit of a path, attention again from the new prefix."""
    cfg = CASES["serving_mix_small"]
    d = torch.device("cuda:0")
    inp = W.make_attn_inputs(cfg, poison=False, capacity_pad=80)
    pk = W.make_paged_cache(inp, 32, salt=9, poison=False)
    paths = W.make_accepted_paths(inp.tree_sizes, inp.tree_parent, cfg.max_tree, cfg.index, 4)
    kd, vd, bt = pk.k_pages.to(d), pk.v_pages.to(d), pk.block_table.to(d)
    new_len, _ = E.eagle_tree_commit_paged(kd, vd, bt, inp.seq_lens.to(d), paths.to(d), cfg.max_tree)
    # next step: a tree of the same shape hangs off the new prefix; its keys are whatever the slots hold (all finite here)
    fits = (new_len.cpu() + inp.tree_sizes) <= (torch.tensor([(int(l) + int(n) + 31) // 32 * 32 for l, n in zip(inp.seq_lens, inp.tree_sizes)]))
    sizes = torch.where(fits, inp.tree_sizes, torch.zeros_like(inp.tree_sizes))
    q = inp.q.clone()
    for b in range(cfg.batch):
        q[b, int(sizes[b]):] = 0
    out = E.eagle_tree_verify_attn_paged(q.to(d), kd, vd, bt, new_len, inp.tree_parent.to(d), tree_sizes=sizes.to(d))
    torch.cuda.synchronize()
    ref = oracle.tree_verify_attn_paged(q, kd.cpu(), vd.cpu(), pk.block_table, new_len.cpu(), inp.tree_parent, sizes)
    _check(out.cpu(), ref, sizes)
