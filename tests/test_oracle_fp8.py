"""Pins of the oracle's fp8 (e4m3) cache form: the code table against a library's conversion, equality with the bf16
oracle on caches whose values are e4m3 numbers, and what the scales must do."""
import numpy as np
import torch

from paper_2401_15077_b200 import workloads as W


def test_e4m3_table_matches_library_conversion(oracle):
    table = oracle.e4m3_table()
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.isnan(table[0x7F]) and np.isnan(table[0xFF]) and np.isnan(lib[0x7F]) and np.isnan(lib[0xFF])
    ok = ~np.isnan(lib)
    assert ok.sum() == 254 and np.array_equal(table[ok], lib[ok])
    assert table[0x7E] == 448.0 and table[0x01] == 2.0 ** -9 and table[0x08] == 2.0 ** -6 and table[0x80] == 0.0
    assert np.signbit(table[0x80]) and table[0x38] == 1.0 and table[0xB8] == -1.0


CFG = W.scaled(W.CONFIGS["tiny"], batch=3, num_q_heads=8, num_kv_heads=2, head_dim=64, prefix=(5, 200), tree=(1, 12))


def test_equals_bf16_oracle_when_values_are_e4m3_numbers(oracle):
    """Every e4m3 number is a bf16 number: the dequantised cache written out as bf16 gives the identical result."""
    inp = W.make_attn_inputs(CFG, salt=1)
    f8 = W.make_fp8_cache(inp, power_of_two_scales=True)          # scales 2^k: code value * scale is still a bf16 number
    table = torch.from_numpy(np.nan_to_num(oracle.e4m3_table(), nan=0.0)).float()
    k = (table[f8.k_codes.long()] * f8.k_scale[:, :, None, None]).to(torch.bfloat16)
    v = (table[f8.v_codes.long()] * f8.v_scale[:, :, None, None]).to(torch.bfloat16)
    assert torch.equal(k.float(), table[f8.k_codes.long()] * f8.k_scale[:, :, None, None])     # nothing was rounded
    a = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, f8.v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    b = oracle.tree_verify_attn(inp.q, k, v, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    assert np.array_equal(a, b)
    # and it is close to the unquantised cache's result (e4m3 keeps 4 significant bits)
    c = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    assert 1e-4 < np.abs(a - c).max() < 0.3


def test_scales(oracle):
    inp = W.make_attn_inputs(CFG, salt=2)
    f8 = W.make_fp8_cache(inp)
    args = (inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    base = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, f8.v_scale, *args, sm_scale=0.125)
    # keys scaled by 4 and the softmax scale by 1/4: the same scores (powers of two: exactly)
    same = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale * 4, f8.v_scale, *args, sm_scale=0.125 / 4)
    assert np.array_equal(base, same)
    # values scaled per (sequence, KV head): the output rows of that head's group scale with it
    vs = f8.v_scale.clone()
    vs[1, 0] *= 2
    twice = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, vs, *args, sm_scale=0.125)
    G = CFG.num_q_heads // CFG.num_kv_heads
    assert np.array_equal(twice[1, :, :G], 2 * base[1, :, :G]) and np.array_equal(twice[1, :, G:], base[1, :, G:])
    assert np.array_equal(twice[0], base[0])
    # slots past prefix + tree hold the NaN code and change nothing; a visible NaN code does
    short = int((inp.seq_lens + inp.tree_sizes).argmin())
    assert np.isfinite(base).all() and (f8.k_codes[short, 0, -1] == 0x7F).all()
    bad = f8.k_codes.clone()
    bad[0, 0, 0, 0] = 0x7F
    assert np.isnan(oracle.tree_verify_attn_fp8(inp.q, bad, f8.v_codes, f8.k_scale, f8.v_scale, *args)[0, 0, 0]).all()


# ---- the fp8 cache kept in pages

def _paged_case(salt, page_size):
    inp = W.make_attn_inputs(CFG, salt=salt)
    f8 = W.make_fp8_cache(inp)
    return inp, f8, W.make_paged_cache(inp, page_size, salt=salt, codes=f8)


def test_paged_fp8_matches_numpy_definition(oracle):
    """An independent evaluation that reads the pages through the table itself and decodes with the library's conversion."""
    page_size = 16
    inp, f8, pk = _paged_case(4, page_size)
    got = oracle.tree_verify_attn_fp8_paged(inp.q, pk.k_pages, pk.v_pages, f8.k_scale, f8.v_scale, pk.block_table, inp.seq_lens,
                                            inp.tree_parent, inp.tree_sizes)
    q = inp.q.to(torch.float64).numpy()
    kp = pk.k_pages.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    vp = pk.v_pages.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    G = CFG.num_q_heads // CFG.num_kv_heads
    for b in range(CFG.batch):
        L, n = int(inp.seq_lens[b]), int(inp.tree_sizes[b])
        for i in range(CFG.max_tree):
            for h in range(CFG.num_q_heads):
                if i >= n:
                    assert np.all(got[b, i, h] == 0.0)
                    continue
                slots = list(range(L))
                c = i
                while c >= 0:
                    slots.append(L + c)
                    c = int(inp.tree_parent[b, c])
                pages = [int(pk.block_table[b, j // page_size]) for j in slots]
                rows = [j % page_size for j in slots]
                K = kp[pages, h // G, rows] * float(f8.k_scale[b, h // G])
                V = vp[pages, h // G, rows] * float(f8.v_scale[b, h // G])
                s = K @ q[b, i, h] / np.sqrt(CFG.head_dim)
                w = np.exp(s - s.max())
                np.testing.assert_allclose(got[b, i, h], (w / w.sum()) @ V, rtol=1e-12, atol=1e-13)


def test_paged_fp8_equals_contiguous_fp8_and_ignores_page_placement(oracle):
    outs = []
    for salt, page_size in ((5, 8), (5, 128), (6, 32)):
        inp, f8, pk = _paged_case(5, page_size)
        pk = W.make_paged_cache(inp, page_size, salt=salt, spare_pages=salt, codes=f8)
        outs.append(oracle.tree_verify_attn_fp8_paged(inp.q, pk.k_pages, pk.v_pages, f8.k_scale, f8.v_scale, pk.block_table,
                                                      inp.seq_lens, inp.tree_parent, inp.tree_sizes))
    flat = oracle.tree_verify_attn_fp8(inp.q, f8.k_codes, f8.v_codes, f8.k_scale, f8.v_scale, inp.seq_lens, inp.tree_parent, inp.tree_sizes)
    assert all(np.array_equal(o, flat) for o in outs)
    # a visible slot without a page is an argument error
    bad = pk.block_table.clone()
    bad[1, 0] = pk.k_pages.shape[0]
    try:
        oracle.tree_verify_attn_fp8_paged(inp.q, pk.k_pages, pk.v_pages, f8.k_scale, f8.v_scale, bad, inp.seq_lens, inp.tree_parent,
                                          inp.tree_sizes)
        raise AssertionError("accepted a page outside the pool")
    except ValueError:
        pass
