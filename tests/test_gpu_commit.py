"""Bit-exact parity of the CUDA commit of the accepted path (through the C ABI) with the oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_2401_15077_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def E():
    from paper_2401_15077_b200 import build, binding
    build.build()
    binding.load()
    assert torch.cuda.is_available()
    return binding


def _bits(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def _run_and_compare(E, oracle, k, v, lens, paths, T, feats=None, expect_status=0):
    d = torch.device("cuda:0")
    ref = oracle.tree_commit(k, v, lens, paths, T, features=feats)
    kd, vd = k.to(d), v.to(d)
    status = torch.zeros(1, dtype=torch.int32, device=d)
    new_len, fout = E.eagle_tree_commit(kd, vd, lens.to(d), paths.to(d), T, features=None if feats is None else feats.to(d),
                                        status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == expect_status
    assert np.array_equal(_bits(kd), ref["k_cache"]) and np.array_equal(_bits(vd), ref["v_cache"])
    assert np.array_equal(new_len.cpu().numpy(), ref["new_seq_lens"])
    if feats is not None:
        assert np.array_equal(_bits(fout), ref["features_out"])
    return ref


CASES = {
    "tiny": (W.CONFIGS["tiny"], 64),
    "7b_mha": (W.CONFIGS["7b_mha"], 4096),
    "70b_gqa": (W.CONFIGS["70b_gqa"], 8192),
    "mix_small": (W.scaled(W.CONFIGS["serving_mix"], batch=12, prefix=(0, 700)), 4096),
    "d64_deep_chains": (W.scaled(W.CONFIGS["tiny"], batch=9, num_q_heads=6, num_kv_heads=3, prefix=(0, 90), tree=(40, 64), max_depth=64,
                                 child_cap=2), 264),
}


@pytest.mark.parametrize("name", list(CASES))
def test_commit_matches_oracle(E, oracle, name):
    cfg, F = CASES[name]
    moved = 0
    for salt in range(3):
        inp = W.make_attn_inputs(cfg, salt=salt, poison=False, capacity_pad=5)
        paths = W.make_accepted_paths(inp.tree_sizes, inp.tree_parent, cfg.max_tree, cfg.index, salt)
        g = torch.Generator().manual_seed(W.seed_for(cfg.index, "features", salt))
        feats = torch.randn((cfg.batch, cfg.max_tree, F), generator=g).to(torch.bfloat16)
        ref = _run_and_compare(E, oracle, inp.k_cache, inp.v_cache, inp.seq_lens, paths, cfg.max_tree, feats)
        assert ref["valid"].all()
        moved += int((ref["new_seq_lens"] - inp.seq_lens.numpy()).sum())
    assert moved > 0


def test_full_size_mix_in_the_bench_configuration(E, oracle):
    cfg = W.CONFIGS["serving_mix"]
    inp = W.make_attn_inputs(cfg, poison=False)
    paths = W.make_accepted_paths(inp.tree_sizes, inp.tree_parent, cfg.max_tree, cfg.index)
    _run_and_compare(E, oracle, inp.k_cache, inp.v_cache, inp.seq_lens, paths, cfg.max_tree)


def test_edge_cases_empty_full_and_long_rows(E, oracle):
    """No accepted node; all 64 nodes of a chain tree; a path row wider than the tree; K only."""
    T, Hkv, D = 64, 2, 128
    g = torch.Generator().manual_seed(5)
    lens = torch.tensor([0, 3, 130, 7], dtype=torch.int32)
    k = torch.randn((4, Hkv, 200, D), generator=g).to(torch.bfloat16)
    v = torch.randn((4, Hkv, 200, D), generator=g).to(torch.bfloat16)
    paths = torch.full((4, 70), -1, dtype=torch.int32)
    paths[1, :64] = torch.arange(64, dtype=torch.int32)                     # the whole chain: identity
    paths[2, :5] = torch.tensor([1, 2, 3, 40, 63], dtype=torch.int32)       # overlapping sources and destinations
    paths[3, :3] = torch.tensor([5, 6, 9], dtype=torch.int32)
    ref = _run_and_compare(E, oracle, k, v, lens, paths, T)
    assert ref["new_seq_lens"].tolist() == [0, 67, 135, 10]
    d = torch.device("cuda:0")
    kd = k.to(d)
    new_len, _ = E.eagle_tree_commit(kd, None, lens.to(d), paths.to(d), T)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(kd), ref["k_cache"])


def test_invalid_paths_are_reported_and_left_alone(E, oracle):
    T = 16
    g = torch.Generator().manual_seed(6)
    lens = torch.tensor([4, 4, 4, 4, 40], dtype=torch.int32)
    k = torch.randn((5, 1, 48, 64), generator=g).to(torch.bfloat16)
    v = torch.randn((5, 1, 48, 64), generator=g).to(torch.bfloat16)
    feats = torch.randn((5, T, 16), generator=g).to(torch.bfloat16)
    paths = torch.full((5, T), -1, dtype=torch.int32)
    paths[0, :2] = torch.tensor([3, 2], dtype=torch.int32)      # decreasing
    paths[1, :2] = torch.tensor([0, 16], dtype=torch.int32)     # outside the tree
    paths[2, :3] = torch.tensor([0, 2, 5], dtype=torch.int32)   # fine
    paths[3, :1] = torch.tensor([-3], dtype=torch.int32)        # not a node
    paths[4, :2] = torch.tensor([2, 9], dtype=torch.int32)      # slot 40 + 9 = 49 does not exist
    ref = _run_and_compare(E, oracle, k, v, lens, paths, T, feats, expect_status=-10)
    assert ref["valid"].tolist() == [0, 0, 1, 0, 0]


@pytest.mark.parametrize("paged", [False, True])
def test_commit_of_an_fp8_cache_moves_rows_of_codes(E, paged):
    """A cache of fp8 codes [.., S, 128] uint8 is committed by the same call on its 16-bit view [.., S, 64]: rows are moved
    as bytes.  The expected cache is built here from the codes, slot by slot."""
    d = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["serving_mix"], batch=5, prefix=(0, 300), tree=(0, 40))
    inp = W.make_attn_inputs(cfg, salt=2, poison=False, capacity_pad=3)
    f8 = W.make_fp8_cache(inp, poison=False)
    for salt in range(8):     # a draw in which some accepted path moves rows (a path 0, 1, 2, ... moves nothing)
        paths = W.make_accepted_paths(inp.tree_sizes, inp.tree_parent, cfg.max_tree, cfg.index, salt)
        if any(int(paths[b, j]) > j for b in range(cfg.batch) for j in range(cfg.max_tree)):
            break
    want_k, want_v = f8.k_codes.clone(), f8.v_codes.clone()
    want_len = inp.seq_lens.clone()
    for b in range(cfg.batch):
        L = int(inp.seq_lens[b])
        path = [int(x) for x in paths[b] if int(x) >= 0]
        for j, m in enumerate(path):
            want_k[b, :, L + j] = f8.k_codes[b, :, L + m]
            want_v[b, :, L + j] = f8.v_codes[b, :, L + m]
        want_len[b] = L + len(path)
    assert any(int(paths[b, j]) > j for b in range(cfg.batch) for j in range(cfg.max_tree))
    status = torch.zeros(1, dtype=torch.int32, device=d)
    if not paged:
        kd, vd = f8.k_codes.to(d), f8.v_codes.to(d)
        new_len, _ = E.eagle_tree_commit(kd.view(torch.bfloat16), vd.view(torch.bfloat16), inp.seq_lens.to(d), paths.to(d), cfg.max_tree,
                                         status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(kd.cpu(), want_k) and torch.equal(vd.cpu(), want_v)
    else:
        pk = W.make_paged_cache(inp, 32, salt=4, poison=False, codes=f8)
        kd, vd = pk.k_pages.to(d), pk.v_pages.to(d)
        new_len, _ = E.eagle_tree_commit_paged(kd.view(torch.bfloat16), vd.view(torch.bfloat16), pk.block_table.to(d), inp.seq_lens.to(d),
                                               paths.to(d), cfg.max_tree, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        want = W.make_paged_cache(inp, 32, salt=4, poison=False, codes=W.Fp8KV(want_k, want_v, f8.k_scale, f8.v_scale))
        # compare slot by slot through the table (rows of pages past the old visible range may differ: the committed
        # prefix grew into them only up to the new length)
        for b in range(cfg.batch):
            if int(inp.tree_sizes[b]) == 0:
                continue                     # (the generator gives a sequence without a tree no pages)
            for j in range(int(want_len[b])):
                page, row = int(pk.block_table[b, j // 32]), j % 32
                assert torch.equal(kd[page, :, row].cpu(), want_k[b, :, j]) and torch.equal(vd[page, :, row].cpu(), want_v[b, :, j]), (b, j)
        del want
    assert torch.equal(new_len.cpu(), want_len)
