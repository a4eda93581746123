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
