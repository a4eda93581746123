"""CPU oracle for EAGLE tree verification (test infrastructure, never on the product path).

Thin ctypes loader around ``eagle_oracle.c`` (plain C, fp64).  Only ``tests/``, the smoke check and
``bench.py``'s CPU-baseline legs may import this package; the CUDA library and its Python binding
share no code with it and never import it.

The arithmetic lives in the C file; the functions here only marshal numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "eagle_oracle.c"
_LIB = _HERE / "liboracle.so"
_lib = None
DEC_ACCEPT, DEC_REJECT, DEC_BONUS, DEC_ARGMAX = 0, 1, 2, 3   # kinds of decision in the acceptance walk's trace


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math) into ``oracle/liboracle.so``."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        i32, dbl, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        lib.oracle_tree_ancestors.argtypes = [vp, vp, i32, i32, vp, vp]
        lib.oracle_tree_ancestors.restype = i32
        lib.oracle_tree_verify_attn.argtypes = [i32, i32, i32, i32, i32, i32, vp, dbl, vp, vp, vp, vp, vp, vp]
        lib.oracle_tree_verify_attn.restype = i32
        lib.oracle_tree_verify_attn_paged.argtypes = [i32] * 8 + [vp, dbl] + [vp] * 7
        lib.oracle_tree_verify_attn_paged.restype = i32
        lib.oracle_tree_verify_attn_fp8.argtypes = [i32, i32, i32, i32, i32, i32, vp, dbl] + [vp] * 8
        lib.oracle_tree_verify_attn_fp8.restype = i32
        lib.oracle_tree_verify_attn_fp8_paged.argtypes = [i32] * 8 + [vp, dbl] + [vp] * 9
        lib.oracle_tree_verify_attn_fp8_paged.restype = i32
        lib.oracle_e4m3_table.argtypes = [vp]
        lib.oracle_e4m3_table.restype = None
        lib.oracle_tree_accept.argtypes = [i32, i32, i32, i32] + [vp] * 17
        lib.oracle_tree_accept.restype = i32
        lib.oracle_tree_accept_logits.argtypes = [i32, i32, i32, i32] + [vp] * 7 + [dbl] + [vp] * 10
        lib.oracle_tree_accept_logits.restype = i32
        lib.oracle_tree_expand.argtypes = [i32, i32, i32, i32] + [vp] * 7
        lib.oracle_tree_expand.restype = i32
        lib.oracle_tree_commit.argtypes = [i32] * 6 + [vp] * 4 + [i32] + [vp] * 4
        lib.oracle_tree_commit.restype = i32
        lib.oracle_tree_commit_paged.argtypes = [i32] * 8 + [vp] * 7
        lib.oracle_tree_commit_paged.restype = i32
        lib.oracle_num_threads.restype = i32
        lib.oracle_set_num_threads.argtypes = [i32]
        lib.oracle_set_num_threads.restype = None
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _as(a, dtype):
    if a is None:
        return None
    if hasattr(a, "detach"):  # torch CPU tensor
        import torch
        if a.dtype == torch.bfloat16:
            a = a.contiguous().view(torch.int16)
        a = a.detach().cpu().numpy()
    a = np.ascontiguousarray(a)
    if dtype == np.uint16 and a.dtype == np.int16:
        a = a.view(np.uint16)
    if a.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {a.dtype}")
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    """Threads for the oracle's OpenMP loops from now on (0: the default).  For timing; results do not depend on it."""
    _load().oracle_set_num_threads(int(n))


def tree_ancestors(tree_parent, tree_sizes=None):
    """Ancestor-or-self bit sets (uint64) and depths (int32) by walking parent links."""
    par = _as(tree_parent, np.int32)
    B, T = par.shape
    ts = _as(tree_sizes, np.int32)
    anc = np.zeros((B, T), np.uint64)
    depth = np.zeros((B, T), np.int32)
    rc = _load().oracle_tree_ancestors(_ptr(par), _ptr(ts), B, T, _ptr(anc), _ptr(depth))
    if rc != 0:
        raise ValueError(f"oracle_tree_ancestors failed: {rc}")
    return anc, depth


def tree_verify_attn(q, k_cache, v_cache, seq_lens, tree_parent, tree_sizes=None, sm_scale: float = 0.0):
    """fp64 tree-masked attention.  q/k/v are bf16 (torch tensors, or their uint16 bit patterns).

    q [B, T_max, Hq, D]; k_cache, v_cache [B, Hkv, S_cap, D]; returns float64 [B, T_max, Hq, D].
    """
    qa, ka, va = _as(q, np.uint16), _as(k_cache, np.uint16), _as(v_cache, np.uint16)
    B, T, Hq, D = qa.shape
    Hkv, S = ka.shape[1], ka.shape[2]
    assert ka.shape == va.shape == (B, Hkv, S, D)
    sl, par, ts = _as(seq_lens, np.int32), _as(tree_parent, np.int32), _as(tree_sizes, np.int32)
    assert par.shape == (B, T)
    out = np.zeros((B, T, Hq, D), np.float64)
    rc = _load().oracle_tree_verify_attn(B, Hq, Hkv, D, T, S, _ptr(ts), float(sm_scale), _ptr(qa), _ptr(ka),
                                         _ptr(va), _ptr(sl), _ptr(par), _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle_tree_verify_attn failed: {rc}")
    return out


def tree_verify_attn_paged(q, k_pages, v_pages, block_table, seq_lens, tree_parent, tree_sizes=None, sm_scale: float = 0.0):
    """fp64 tree-masked attention over a paged cache.

    q [B, T_max, Hq, D]; k_pages, v_pages [num_pages, Hkv, page_size, D]; block_table int32 [B, max_pages_per_seq];
    returns float64 [B, T_max, Hq, D].
    """
    qa, ka, va = _as(q, np.uint16), _as(k_pages, np.uint16), _as(v_pages, np.uint16)
    B, T, Hq, D = qa.shape
    P, Hkv, ps = ka.shape[0], ka.shape[1], ka.shape[2]
    assert ka.shape == va.shape == (P, Hkv, ps, D)
    bt = _as(block_table, np.int32)
    assert bt.ndim == 2 and bt.shape[0] == B
    sl, par, ts = _as(seq_lens, np.int32), _as(tree_parent, np.int32), _as(tree_sizes, np.int32)
    assert par.shape == (B, T)
    out = np.zeros((B, T, Hq, D), np.float64)
    rc = _load().oracle_tree_verify_attn_paged(B, Hq, Hkv, D, T, P, ps, bt.shape[1], _ptr(ts), float(sm_scale), _ptr(qa),
                                               _ptr(ka), _ptr(va), _ptr(bt), _ptr(sl), _ptr(par), _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle_tree_verify_attn_paged failed: {rc}")
    return out


def e4m3_table():
    """The 256 values of the fp8 e4m3 codes as the oracle decodes them (float64; the two NaN codes are NaN)."""
    out = np.zeros(256, np.float64)
    _load().oracle_e4m3_table(_ptr(out))
    return out


def tree_verify_attn_fp8(q, k_codes, v_codes, k_scale, v_scale, seq_lens, tree_parent, tree_sizes=None, sm_scale: float = 0.0):
    """fp64 tree-masked attention over a cache stored as e4m3 codes (uint8 [B, Hkv, S_cap, D]) with fp32 scales [B, Hkv]:
    key = code value * k_scale, value = code value * v_scale.  q is bf16.  Returns float64 [B, T_max, Hq, D]."""
    qa = _as(q, np.uint16)
    ka, va = _as(k_codes, np.uint8), _as(v_codes, np.uint8)
    B, T, Hq, D = qa.shape
    Hkv, S = ka.shape[1], ka.shape[2]
    assert ka.shape == va.shape == (B, Hkv, S, D)
    ks, vs = _as(k_scale, np.float32), _as(v_scale, np.float32)
    assert ks.shape == vs.shape == (B, Hkv)
    sl, par, ts = _as(seq_lens, np.int32), _as(tree_parent, np.int32), _as(tree_sizes, np.int32)
    out = np.zeros((B, T, Hq, D), np.float64)
    rc = _load().oracle_tree_verify_attn_fp8(B, Hq, Hkv, D, T, S, _ptr(ts), float(sm_scale), _ptr(qa), _ptr(ka), _ptr(va),
                                             _ptr(ks), _ptr(vs), _ptr(sl), _ptr(par), _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle_tree_verify_attn_fp8 failed: {rc}")
    return out


def tree_verify_attn_fp8_paged(q, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens, tree_parent, tree_sizes=None,
                              sm_scale: float = 0.0):
    """fp64 tree-masked attention over a paged cache of e4m3 codes: k_pages, v_pages uint8 [num_pages, Hkv, page_size, D],
    scales fp32 [B, Hkv], block_table int32 [B, max_pages_per_seq].  Returns float64 [B, T_max, Hq, D]."""
    qa = _as(q, np.uint16)
    ka, va = _as(k_pages, np.uint8), _as(v_pages, np.uint8)
    B, T, Hq, D = qa.shape
    P, Hkv, ps = ka.shape[0], ka.shape[1], ka.shape[2]
    assert ka.shape == va.shape == (P, Hkv, ps, D)
    ks, vs = _as(k_scale, np.float32), _as(v_scale, np.float32)
    assert ks.shape == vs.shape == (B, Hkv)
    bt = _as(block_table, np.int32)
    assert bt.ndim == 2 and bt.shape[0] == B
    sl, par, ts = _as(seq_lens, np.int32), _as(tree_parent, np.int32), _as(tree_sizes, np.int32)
    assert par.shape == (B, T)
    out = np.zeros((B, T, Hq, D), np.float64)
    rc = _load().oracle_tree_verify_attn_fp8_paged(B, Hq, Hkv, D, T, P, ps, bt.shape[1], _ptr(ts), float(sm_scale), _ptr(qa),
                                                   _ptr(ka), _ptr(va), _ptr(ks), _ptr(vs), _ptr(bt), _ptr(sl), _ptr(par), _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle_tree_verify_attn_fp8_paged failed: {rc}")
    return out


def tree_accept(target_probs, draft_probs, draft_tokens, tree_parent, uniforms, tree_sizes=None, greedy=None,
                path_cap: int | None = None, temperature: float | None = None):
    """Acceptance walk (Algorithm 1 at every node, or the greedy rule).  Returns a dict of numpy arrays:
    accepted_path [B, path_cap], bonus_token [B], accept_len [B], min_margin [B], n_sweeps [B],
    n_zero_mass [B], and the walk's decisions in order: n_dec [B], dec_kind / dec_node / dec_margin [B, T+1]
    (kinds: DEC_ACCEPT, DEC_REJECT, DEC_BONUS, DEC_ARGMAX)."""
    tp = _as(target_probs, np.float32)
    B, T1, V = tp.shape
    T = T1 - 1
    dp = _as(draft_probs, np.float32)
    tok, par = _as(draft_tokens, np.int32), _as(tree_parent, np.int32)
    un = _as(uniforms, np.float32)
    ts, gr = _as(tree_sizes, np.int32), _as(greedy, np.uint8)
    assert tok.shape == par.shape == (B, T)
    if dp is not None:
        assert dp.shape == (B, T, V)
    if un is not None:
        assert un.shape == (B, T + 1)
    cap = T if path_cap is None else path_cap
    res = dict(accepted_path=np.full((B, cap), -1, np.int32), bonus_token=np.full((B,), -1, np.int32),
               accept_len=np.zeros((B,), np.int32), min_margin=np.zeros((B,), np.float64),
               n_sweeps=np.zeros((B,), np.int32), n_zero_mass=np.zeros((B,), np.int32),
               n_dec=np.zeros((B,), np.int32), dec_kind=np.full((B, T + 1), -1, np.int32),
               dec_node=np.full((B, T + 1), -2, np.int32), dec_margin=np.full((B, T + 1), np.nan, np.float64))
    trace = (_ptr(res["n_dec"]), _ptr(res["dec_kind"]), _ptr(res["dec_node"]), _ptr(res["dec_margin"]))
    if temperature is None:
        rc = _load().oracle_tree_accept(B, T, V, cap, _ptr(ts), _ptr(gr), _ptr(tp), _ptr(dp), _ptr(tok), _ptr(par),
                                        _ptr(un), _ptr(res["accepted_path"]), _ptr(res["bonus_token"]),
                                        _ptr(res["accept_len"]), _ptr(res["min_margin"]), _ptr(res["n_sweeps"]),
                                        _ptr(res["n_zero_mass"]), *trace)
    else:
        rc = _load().oracle_tree_accept_logits(B, T, V, cap, _ptr(ts), _ptr(gr), _ptr(tp), _ptr(dp), _ptr(tok), _ptr(par),
                                               _ptr(un), float(temperature), _ptr(res["accepted_path"]),
                                               _ptr(res["bonus_token"]), _ptr(res["accept_len"]), _ptr(res["min_margin"]),
                                               _ptr(res["n_sweeps"]), _ptr(res["n_zero_mass"]), *trace)
    if rc != 0:
        raise ValueError(f"oracle_tree_accept failed: {rc}")
    return res


def tree_accept_logits(target_logits, draft_logits, draft_tokens, tree_parent, uniforms, temperature: float,
                       tree_sizes=None, greedy=None, path_cap: int | None = None):
    """The acceptance walk with the distributions given as fp32 logits: rows are softmax(logits / temperature) in fp64."""
    return tree_accept(target_logits, draft_logits, draft_tokens, tree_parent, uniforms, tree_sizes=tree_sizes, greedy=greedy,
                       path_cap=path_cap, temperature=temperature)


def tree_commit(k_cache, v_cache, seq_lens, accepted_path, max_tree: int, features=None):
    """Commit of the accepted path (Sec. 3.3).  ``k_cache`` / ``v_cache``: bf16 [B, Hkv, S_cap, D] (torch CPU tensors
    or uint16 arrays); they are NOT modified: copies are returned.  Returns a dict: k_cache, v_cache (uint16 arrays),
    features_out [B, path_cap, F] (uint16, or None), new_seq_lens [B], valid [B]."""
    k = _as(k_cache, np.uint16).copy()
    v = _as(v_cache, np.uint16).copy()
    sl, path = _as(seq_lens, np.int32), _as(accepted_path, np.int32)
    B, Hkv, S_cap, D = k.shape
    assert v.shape == k.shape and path.shape[0] == B and sl.shape == (B,)
    cap = path.shape[1]
    fin = _as(features, np.uint16)
    F = 0 if fin is None else fin.shape[2]
    if fin is not None:
        assert fin.shape[:2] == (B, max_tree)
    fout = None if fin is None else np.full((B, cap, F), 0xFFFF, np.uint16)
    new_len = np.full((B,), -1, np.int32)
    valid = np.full((B,), -1, np.int32)
    rc = _load().oracle_tree_commit(B, Hkv, D, S_cap, max_tree, cap, _ptr(sl), _ptr(path), _ptr(k), _ptr(v), F, _ptr(fin),
                                    _ptr(fout), _ptr(new_len), _ptr(valid))
    if rc != 0:
        raise ValueError(f"oracle_tree_commit failed: {rc}")
    return dict(k_cache=k, v_cache=v, features_out=fout, new_seq_lens=new_len, valid=valid)


def tree_commit_paged(k_pages, v_pages, block_table, seq_lens, accepted_path, max_tree: int):
    """Commit of the accepted path on a paged cache.  ``k_pages`` / ``v_pages``: bf16 [num_pages, Hkv, page_size, D];
    they are NOT modified: copies are returned.  Returns a dict: k_pages, v_pages (uint16 arrays), new_seq_lens, valid."""
    k = _as(k_pages, np.uint16).copy()
    v = _as(v_pages, np.uint16).copy()
    bt, sl, path = _as(block_table, np.int32), _as(seq_lens, np.int32), _as(accepted_path, np.int32)
    P, Hkv, ps, D = k.shape
    B = sl.shape[0]
    assert v.shape == k.shape and path.shape[0] == B and bt.shape[0] == B
    new_len = np.full((B,), -1, np.int32)
    valid = np.full((B,), -1, np.int32)
    rc = _load().oracle_tree_commit_paged(B, Hkv, D, P, ps, bt.shape[1], max_tree, path.shape[1], _ptr(sl), _ptr(path), _ptr(bt),
                                          _ptr(k), _ptr(v), _ptr(new_len), _ptr(valid))
    if rc != 0:
        raise ValueError(f"oracle_tree_commit_paged failed: {rc}")
    return dict(k_pages=k, v_pages=v, new_seq_lens=new_len, valid=valid)


def tree_expand(probs, num_children, max_children: int, uniforms=None, greedy=None):
    """Child tokens of draft-tree nodes (App. A.1): top-k of each row for greedy sequences, k independent inverse-CDF draws
    otherwise.  probs [B, R, V] fp32, num_children [B, R] int32, uniforms [B, R, max_children] fp32, greedy [B] uint8.
    Returns a dict: tokens [B, R, max_children] int32 (-1 padded), token_probs fp32, min_margin [B, R]."""
    p = _as(probs, np.float32)
    B, R, V = p.shape
    nc, un, gr = _as(num_children, np.int32), _as(uniforms, np.float32), _as(greedy, np.uint8)
    assert nc.shape == (B, R) and (un is None or un.shape == (B, R, max_children))
    res = dict(tokens=np.full((B, R, max_children), -2, np.int32), token_probs=np.full((B, R, max_children), -1, np.float32),
               min_margin=np.zeros((B, R), np.float64))
    rc = _load().oracle_tree_expand(B, R, V, max_children, _ptr(nc), _ptr(gr), _ptr(p), _ptr(un), _ptr(res["tokens"]),
                                    _ptr(res["token_probs"]), _ptr(res["min_margin"]))
    if rc != 0:
        raise ValueError(f"oracle_tree_expand failed: {rc}")
    return res
