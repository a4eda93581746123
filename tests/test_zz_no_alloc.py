"""The workspace-free attention entry point (collected last on purpose: it shares one fixed device array per GPU).

``eagle_tree_verify_attn_static`` is for hosts that can pass device tensors but cannot obtain device scratch when
they run (a serving backend with a frozen memory pool, a plug-in inside another engine's context, a decode loop that
must not call cudaMalloc).  It must give what ``eagle_tree_verify_attn`` gives, call after call, although every
call reuses the same array and finds the previous call's plan and partials in it.
"""
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


def _dev(inp):
    d = torch.device("cuda:0")
    return dict(q=inp.q.to(d), k=inp.k_cache.to(d), v=inp.v_cache.to(d), sl=inp.seq_lens.to(d),
                par=inp.tree_parent.to(d), ts=inp.tree_sizes.to(d))


def test_static_entry_matches_workspace_entry_twice_in_a_row(E, oracle):
    assert E.static_capacity() == 24 << 20
    # two different problems back to back, so that the second call finds the first one's leftovers in the array:
    # a ragged batch that gets cut into partials, then a smaller one with another head layout
    cases = [W.scaled(W.CONFIGS["serving_mix"], batch=6, prefix=(100, 3000), tree=(5, 64)),
             W.scaled(W.CONFIGS["tiny"], batch=3, num_q_heads=16, num_kv_heads=4, prefix=(0, 900), tree=(1, 20))]
    for rep, cfg in enumerate(cases + cases[:1]):
        t = _dev(W.make_attn_inputs(cfg, salt=rep))
        status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        want = torch.full_like(t["q"], float("nan"))
        E.eagle_tree_verify_attn(t["q"], t["k"], t["v"], t["sl"], t["par"], want, tree_sizes=t["ts"], status=status)
        got = torch.full_like(t["q"], float("nan"))
        if rep == 0:    # the first call on a device looks up the array's address; later calls must not touch any allocator
            E.eagle_tree_verify_attn_static(t["q"], t["k"], t["v"], t["sl"], t["par"], got, tree_sizes=t["ts"], status=status)
            torch.cuda.synchronize()
        before, free_before, launches = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0], E.launch_count()
        E.eagle_tree_verify_attn_static(t["q"], t["k"], t["v"], t["sl"], t["par"], got, tree_sizes=t["ts"], status=status)
        assert torch.cuda.memory_allocated() == before      # nothing was taken from torch's allocator
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before    # nor from the device behind torch's back (cudaMemGetInfo)
        assert E.launch_count() == launches + 3               # planner, attention, combine
        assert int(status.item()) == 0
        a, b = got.cpu().double().numpy(), want.cpu().double().numpy()
        assert np.isfinite(a).all()
        # the two entry points run the same kernels; their work split may differ (the fixed array is carved for this
        # GPU's SM count), so partial sums can associate differently: same bounds as against the oracle
        assert np.abs(a - b).max() <= 2e-2 and np.abs(a - b).mean() <= 2e-3
        # and against the oracle itself
        inp = W.make_attn_inputs(cfg, salt=rep)
        ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
        rows = np.zeros(ref.shape[:2], bool)
        for i, n in enumerate(inp.tree_sizes):
            rows[i, :int(n)] = True
        err = np.abs(a - ref)
        assert err[rows].max() <= 2e-2 and err[rows].mean() <= 2e-3 and np.all(a[~rows] == 0.0)


def test_static_entry_takes_the_full_batched_configuration(E, oracle):
    """The 64-sequence serving mix (512 work units, most CTA shares cutting one) fits the fixed array: its partials are
    bounded by the number of CTAs, not by the batch.  Sampled (sequence, KV head) units are checked against the oracle."""
    cfg = W.CONFIGS["serving_mix"]
    inp = W.make_attn_inputs(cfg)
    t = _dev(inp)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    got = torch.full_like(t["q"], float("nan"))
    E.eagle_tree_verify_attn_static(t["q"], t["k"], t["v"], t["sl"], t["par"], got, tree_sizes=t["ts"], status=status)
    want = torch.full_like(t["q"], float("nan"))
    E.eagle_tree_verify_attn(t["q"], t["k"], t["v"], t["sl"], t["par"], want, tree_sizes=t["ts"], status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    a = got.cpu().double().numpy()
    assert np.isfinite(a).all() and np.abs(a - want.cpu().double().numpy()).max() <= 2e-2
    G = cfg.num_q_heads // cfg.num_kv_heads
    for b, g in [(int(inp.seq_lens.argmax()), 0), (int(inp.seq_lens.argmin()), 7), (17, 3)]:
        n, end = int(inp.tree_sizes[b]), int(inp.seq_lens[b] + inp.tree_sizes[b])
        ref = oracle.tree_verify_attn(inp.q[b:b + 1, :, g * G:(g + 1) * G].contiguous(), inp.k_cache[b:b + 1, g:g + 1, :end].contiguous(),
                                      inp.v_cache[b:b + 1, g:g + 1, :end].contiguous(), inp.seq_lens[b:b + 1], inp.tree_parent[b:b + 1],
                                      inp.tree_sizes[b:b + 1])
        err = np.abs(a[b, :n, g * G:(g + 1) * G] - ref[0, :n])
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (b, g, err.max())


def test_static_entry_refuses_what_does_not_fit(E):
    cfg = W.scaled(W.CONFIGS["tiny"], batch=2)
    t = _dev(W.make_attn_inputs(cfg))
    out = torch.zeros_like(t["q"])
    # forcing 64 splits of every unit of a large batch needs far more partial slots than the fixed array holds
    big = W.scaled(W.CONFIGS["70b_gqa"], batch=64, prefix=(10, 10), tree=(60, 60))
    tb = _dev(W.make_attn_inputs(big))
    with pytest.raises(E.EagleError, match="workspace"):
        E.eagle_tree_verify_attn_static(tb["q"], tb["k"], tb["v"], tb["sl"], tb["par"], torch.zeros_like(tb["q"]),
                                        tree_sizes=tb["ts"], num_splits=64)
    # and the array is still usable afterwards
    E.eagle_tree_verify_attn_static(t["q"], t["k"], t["v"], t["sl"], t["par"], out, tree_sizes=t["ts"])
    torch.cuda.synchronize()
    assert torch.isfinite(out[:, :8].float()).all()
