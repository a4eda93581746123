"""The C-ABI library builds, loads without a GPU, exports what include/eagle_verify.h declares, and its
host-side argument checks answer before anything is launched."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2401_15077_b200 import build, binding
    build.build()
    return binding.load()


def test_every_declared_symbol_is_exported(lib):
    from paper_2401_15077_b200 import binding
    header = (ROOT / "include" / "eagle_verify.h").read_text()
    declared = set(re.findall(r"\b(eagle_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    from paper_2401_15077_b200 import binding
    assert binding.status_string(0) == "ok"
    seen = {binding.status_string(c) for c in range(-11, 1)}
    assert len(seen) == 12 and "unknown status" not in seen
    assert binding.status_string(-1234) == "unknown status"


def test_workspace_query_and_shape_checks(lib):
    from paper_2401_15077_b200 import binding
    n = binding.eagle_tree_verify_attn_workspace(4, 64, 8, 128, 60)
    assert n > 0 and n % 256 == 0
    # forced splits need (units * splits) partial slots
    assert binding.eagle_tree_verify_attn_workspace(4, 64, 8, 128, 60, num_splits=4) > 0
    assert binding.eagle_tree_verify_attn_workspace(1, 8, 8, 64, 8, num_splits=1) < n
    for bad in [dict(head_dim=96), dict(num_q_heads=12, num_kv_heads=8), dict(max_tree=65), dict(num_q_heads=64, num_kv_heads=2)]:
        kw = dict(batch=1, num_q_heads=8, num_kv_heads=8, head_dim=64, max_tree=8)
        kw.update(bad)
        with pytest.raises(binding.EagleError):
            binding.eagle_tree_verify_attn_workspace(**kw)


def test_host_checks_return_before_any_launch(lib):
    from paper_2401_15077_b200 import binding
    before = binding.launch_count()
    assert lib.eagle_tree_verify_attn(None, None, None, None, None, None, None, None) == -1
    d = binding.AttnDesc(1, 8, 8, 64, 8, 300, None, 0.0, 0, None, 0, None, None, None)
    # null tensors
    assert lib.eagle_tree_verify_attn(ctypes.byref(d), None, None, None, None, None, None, None) == -1
    # batch 0 is a no-op
    d0 = binding.AttnDesc(0, 8, 8, 64, 8, 300, None, 0.0, 0, None, 0, None, None, None)
    assert lib.eagle_tree_verify_attn(ctypes.byref(d0), None, None, None, None, None, None, None) == 0
    # non-null tensors but no workspace
    fake = ctypes.c_void_p(4096)
    assert lib.eagle_tree_verify_attn(ctypes.byref(d), fake, fake, fake, fake, fake, fake, None) == -3
    # a workspace that would do, but an output that is not 32-byte aligned (or a query that is not 16-byte aligned)
    dws = binding.AttnDesc(1, 8, 8, 64, 8, 300, None, 0.0, 0, 4096, 1 << 30, None, None, None)
    assert lib.eagle_tree_verify_attn(ctypes.byref(dws), fake, fake, fake, fake, fake, ctypes.c_void_p(4096 + 16), None) == -2
    assert lib.eagle_tree_verify_attn(ctypes.byref(dws), ctypes.c_void_p(4096 + 8), fake, fake, fake, fake, fake, None) == -2
    dbad = binding.AttnDesc(1, 8, 8, 80, 8, 300, None, 0.0, 0, None, 0, None, None, None)
    assert lib.eagle_tree_verify_attn(ctypes.byref(dbad), fake, fake, fake, fake, fake, fake, None) == -2
    a = binding.AcceptDesc(1, 65, 10, 8, None, None, None, None)
    assert lib.eagle_tree_accept(ctypes.byref(a), fake, fake, fake, fake, fake, fake, fake, None) == -2
    a = binding.AcceptDesc(1, 8, 10, 8, None, None, None, None)
    assert lib.eagle_tree_accept(ctypes.byref(a), None, fake, fake, fake, fake, fake, fake, None) == -1
    assert lib.eagle_tree_accept(ctypes.byref(a), fake, None, fake, fake, fake, fake, fake, None) == -1
    assert lib.eagle_tree_build_mask(None, None, 1, 8, None, None, None, None) == -1
    assert lib.eagle_tree_build_mask(fake, None, 1, 99, fake, None, None, None) == -2
    # paged cache: descriptor checks come first
    assert lib.eagle_tree_verify_attn_paged(ctypes.byref(d), fake, None, fake, fake, fake, None) == -1
    for pages, size, per_seq, want in [(0, 16, 4, -2), (4, 8, 4, -2), (4, 48, 4, -2), (4, 16, -1, -2), (4, 16, 4, -3)]:
        pk = binding.PagedKV(4096, 4096, 4096, pages, size, per_seq)
        assert lib.eagle_tree_verify_attn_paged(ctypes.byref(d), fake, ctypes.byref(pk), fake, fake, fake, None) == want
    pk = binding.PagedKV(4096, 4096, None, 4, 16, 4)
    assert lib.eagle_tree_verify_attn_paged(ctypes.byref(d), fake, ctypes.byref(pk), fake, fake, fake, None) == -1
    c = binding.CommitDesc(1, 8, 64, 0, 8, 8, 0, None)
    assert lib.eagle_tree_commit_paged(ctypes.byref(c), None, fake, fake, None, None, None, None) == -1
    pk = binding.PagedKV(4096, 4096, 4096, 4, 24, 4)
    assert lib.eagle_tree_commit_paged(ctypes.byref(c), ctypes.byref(pk), fake, fake, None, None, None, None) == -2
    # the entry points added for the steps around verification: same rules
    assert lib.eagle_tree_accept_logits(ctypes.byref(a), fake, fake, fake, fake, fake, ctypes.c_float(0.0), fake, fake, None) == -2
    assert lib.eagle_tree_accept_logits(ctypes.byref(a), fake, fake, fake, fake, fake, ctypes.c_float(float("nan")), fake, fake, None) == -2
    assert lib.eagle_tree_accept_logits(ctypes.byref(a), None, fake, fake, fake, fake, ctypes.c_float(1.0), fake, fake, None) == -1
    c = binding.CommitDesc(2, 4, 128, 512, 64, 64, 0, None)
    assert lib.eagle_tree_commit(None, fake, fake, fake, fake, None, None, None, None) == -1
    assert lib.eagle_tree_commit(ctypes.byref(c), fake, fake, None, fake, None, None, None, None) == -1
    assert lib.eagle_tree_commit(ctypes.byref(c), ctypes.c_void_p(4100), fake, fake, fake, None, None, None, None) == -2   # misaligned cache
    for bad in (binding.CommitDesc(2, 4, 96, 512, 64, 64, 0, None), binding.CommitDesc(2, 4, 128, 512, 65, 64, 0, None),
                binding.CommitDesc(2, 4, 128, 512, 64, 64, 12, None)):
        assert lib.eagle_tree_commit(ctypes.byref(bad), fake, fake, fake, fake, None, None, None, None) == -2
    assert lib.eagle_tree_commit(ctypes.byref(binding.CommitDesc(0, 4, 128, 512, 64, 64, 0, None)), None, None, None, None, None, None,
                                 None, None) == 0
    e = binding.ExpandDesc(2, 3, 100, 4, None, None)
    assert lib.eagle_tree_expand(ctypes.byref(e), None, fake, fake, fake, None, None) == -1
    assert lib.eagle_tree_expand(ctypes.byref(e), fake, fake, None, fake, None, None) == -1            # stochastic rows need uniforms
    assert lib.eagle_tree_expand(ctypes.byref(binding.ExpandDesc(2, 3, 100, 17, None, None)), fake, fake, fake, fake, None, None) == -2
    assert lib.eagle_tree_expand(ctypes.byref(binding.ExpandDesc(2, 0, 100, 4, None, None)), None, None, None, None, None, None) == 0
    assert binding.launch_count() == before


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2401_15077_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(binding.EagleError):
        binding.load()


def test_host_step_byte_count(lib):
    """eagle_tree_verify_step_host_bytes: whole tensors when trimming would not pay, else only the visible cache slots and the
    rows of existing nodes (counted here from the same host arrays)."""
    import numpy as np
    from paper_2401_15077_b200 import binding
    B, Hq, Hkv, D, T, S, V = 6, 8, 2, 64, 16, 4000, 2048
    fake = 4096

    def make(lens, sizes):
        s = binding.HostStep()
        s.batch, s.num_q_heads, s.num_kv_heads, s.head_dim, s.max_tree = B, Hq, Hkv, D, T
        s.kv_capacity, s.vocab, s.path_cap, s.sm_scale = S, V, T, 0.0
        for name in ("q", "k_cache", "v_cache", "tree_parent", "target_probs", "draft_probs", "draft_tokens", "uniforms", "greedy"):
            setattr(s, name, fake)
        s.seq_lens, s.tree_sizes = lens.ctypes.data, sizes.ctypes.data
        h2d, d2h = ctypes.c_size_t(0), ctypes.c_size_t(0)
        assert lib.eagle_tree_verify_step_host_bytes(ctypes.byref(s), ctypes.byref(h2d), ctypes.byref(d2h)) == 0
        return h2d.value, d2h.value

    small = B * T * Hq * D * 2 + 2 * B * 4 + 2 * B * T * 4 + B * (T + 1) * 4 + B
    full = small + 2 * B * Hkv * S * D * 2 + B * (T + 1) * V * 4 + B * T * V * 4
    d2h_want = B * T * Hq * D * 2 + B * T * 4 + 2 * B * 4 + 4
    # every sequence fills the cache and the tree: nothing to save
    lens, sizes = np.full(B, S - T, np.int32), np.full(B, T, np.int32)
    assert make(lens, sizes) == (full, d2h_want)
    # ragged: visible slots and existing rows only; an empty tree reads nothing of its cache; bad lengths are clamped
    lens = np.array([100, 3000, 0, 2500, -5, 50], np.int32)
    sizes = np.array([16, 3, 7, 0, 9, 99], np.int32)
    want = small
    for L, n in zip(lens, sizes):
        n = min(max(int(n), 0), T)
        vis = min(max(int(L) + n, 0), S) if n > 0 else 0
        want += 2 * vis * Hkv * D * 2 + (n + 1) * V * 4 + n * V * 4
    assert want < full
    assert make(lens, sizes) == (want, d2h_want)
    assert lib.eagle_tree_verify_step_host_bytes(None, None, None) == -1


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: the header compiles as C99 with warnings as errors, without CUDA or C++."""
    import subprocess
    src = tmp_path / "use_header.c"
    src.write_text('#include "eagle_verify.h"\n'
                   'int main(void) { eagle_attn_desc d; eagle_accept_desc a; eagle_paged_kv k; (void)d; (void)a; (void)k;\n'
                   '  return sizeof(eagle_host_step) > 0 && EAGLE_MAX_TREE == 64 ? 0 : 1; }\n')
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-fsyntax-only", "-I", str(ROOT / "include"), str(src)],
                   check=True)
