"""The drafting phase as a loop (App. A.1: the draft tree grows over five passes, every node getting k children):
tree attention on the partial tree, child selection on the new nodes' draft rows, append, repeat; then verification of
the finished tree.

CPU part (pins the oracle's partial-tree semantics, what `tree_sizes` means): a node sees the prefix, its ancestors and
itself, all of which were appended before it, so its attention row never changes when later nodes are appended: every
pass's rows equal the finished tree's rows.  GPU part: the same loop through the C ABI, every pass against the oracle.
"""
import numpy as np
import pytest
import torch

from paper_2401_15077_b200 import workloads as W

PASSES, K_CHILD, T_MAX = 5, 2, 40


def _draft_rows(seed, B, n_rows, V):
    """Synthetic draft distributions of the nodes expanded in one pass (there is no draft model here)."""
    g = torch.Generator().manual_seed(seed)
    return torch.softmax(torch.randn((B, n_rows, V), generator=g) * 1.4142, dim=-1)


def _grow(oracle, expand, attend, B, V, greedy, cfg, seed):
    """Runs the loop.  ``expand(probs, nc, un)`` -> child tokens [B, R, K]; ``attend(sizes)`` -> rows for the current
    partial tree.  Returns the per-pass attention rows, the final parents / sizes, and the token of every node."""
    parent = torch.full((B, T_MAX), 2 ** 30, dtype=torch.int32)      # entries of nodes that do not exist yet are never read
    tokens = torch.zeros((B, T_MAX), dtype=torch.int32)
    sizes = torch.zeros(B, dtype=torch.int32)
    frontier = [[-1] for _ in range(B)]                                # nodes expanded in the next pass (-1: the context)
    per_pass = []
    for d in range(PASSES):
        R = max(len(f) for f in frontier)
        nc = torch.zeros((B, R), dtype=torch.int32)
        for b in range(B):
            for j, node in enumerate(frontier[b]):
                room = T_MAX - int(sizes[b]) - int(nc[b].sum())
                nc[b, j] = max(0, min(K_CHILD if d else 4, room))      # four children of the context, then k per node
        probs = _draft_rows(seed * 100 + d, B, R, V)
        un = torch.rand((B, R, 4), generator=torch.Generator().manual_seed(seed * 100 + 50 + d))
        child = expand(probs, nc, un)
        new_frontier = []
        for b in range(B):
            nf = []
            for j, node in enumerate(frontier[b]):
                for c in range(int(nc[b, j])):
                    i = int(sizes[b])
                    parent[b, i], tokens[b, i] = node, int(child[b, j, c])
                    sizes[b] += 1
                    nf.append(i)
            new_frontier.append(nf[:4])                                 # expand at most four nodes of a level
        frontier = new_frontier
        per_pass.append((sizes.clone(), attend(parent, sizes)))
    return per_pass, parent, sizes, tokens


def _inputs(cfg):
    inp = W.make_attn_inputs(cfg, salt=21)
    # the tree's K/V rows of every slot up to T_MAX are filled in advance: node m's rows wait at slot L + m
    g = torch.Generator().manual_seed(77)
    for b in range(cfg.batch):
        L = int(inp.seq_lens[b])
        inp.k_cache[b, :, L:L + T_MAX] = torch.randn((cfg.num_kv_heads, T_MAX, cfg.head_dim), generator=g).to(torch.bfloat16)
        inp.v_cache[b, :, L:L + T_MAX] = torch.randn((cfg.num_kv_heads, T_MAX, cfg.head_dim), generator=g).to(torch.bfloat16)
    inp.q = torch.randn(inp.q.shape, generator=g).to(torch.bfloat16)
    return inp


CFG = W.scaled(W.CONFIGS["tiny"], batch=3, num_q_heads=8, num_kv_heads=2, head_dim=128, prefix=(90, 300), tree=(T_MAX, T_MAX))


def test_oracle_rows_of_a_growing_tree_never_change(oracle):
    inp = _inputs(CFG)
    V, greedy = 500, torch.tensor([1, 0, 1], dtype=torch.uint8)

    def expand(probs, nc, un):
        return oracle.tree_expand(probs, nc, 4, uniforms=un, greedy=greedy)["tokens"]

    def attend(parent, sizes):
        return oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, parent.clone(), sizes.clone())

    per_pass, parent, sizes, tokens = _grow(oracle, expand, attend, CFG.batch, V, greedy, CFG, seed=3)
    assert int(sizes.min()) > 15 and int(sizes.max()) <= T_MAX
    anc, depth = oracle.tree_ancestors(parent.numpy(), sizes.numpy())
    assert depth.max() == PASSES                                         # five passes -> five levels
    final = per_pass[-1][1]
    for n_then, rows in per_pass:
        for b in range(CFG.batch):
            n = int(n_then[b])
            assert np.array_equal(rows[b, :n], final[b, :n])             # exactly: the same visible set, the same arithmetic
            assert np.all(rows[b, n:] == 0.0)
    # greedy sequences: the children of a node are its row's top tokens in rank order, so siblings carry distinct tokens
    for b in (0, 2):
        for p in set(parent[b, :int(sizes[b])].tolist()):
            sib = [int(tokens[b, i]) for i in range(int(sizes[b])) if int(parent[b, i]) == p]
            assert len(set(sib)) == len(sib)


@pytest.mark.gpu
def test_drafting_loop_on_gpu_matches_oracle(oracle):
    from paper_2401_15077_b200 import build, binding as E
    build.build()
    E.load()
    d = torch.device("cuda:0")
    inp = _inputs(CFG)
    V, greedy = 500, torch.tensor([1, 0, 1], dtype=torch.uint8)
    q, k, v, sl = inp.q.to(d), inp.k_cache.to(d), inp.v_cache.to(d), inp.seq_lens.to(d)
    status = torch.zeros(1, dtype=torch.int32, device=d)
    seen = {"expand_rows": 0}

    def expand(probs, nc, un):
        ref = oracle.tree_expand(probs, nc, 4, uniforms=un, greedy=greedy)
        tok, _ = E.eagle_tree_expand(probs.to(d), nc.to(d), 4, uniforms=un.to(d), greedy=greedy.to(d), status=status)
        torch.cuda.synchronize()
        tok = tok.cpu().numpy()
        for b in range(nc.shape[0]):
            for r in range(nc.shape[1]):
                assert np.array_equal(tok[b, r], ref["tokens"][b, r]) or (not greedy[b] and ref["min_margin"][b, r] < 1e-9)
                seen["expand_rows"] += 1
        return ref["tokens"]          # the tree follows the oracle's choice (identical unless a draw sat on a cell edge)

    def attend(parent, sizes):
        out = torch.full_like(q, float("nan"))
        E.eagle_tree_verify_attn(q, k, v, sl, parent.to(d), out, tree_sizes=sizes.to(d), status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = out.cpu().double().numpy()
        ref = oracle.tree_verify_attn(inp.q, inp.k_cache, inp.v_cache, inp.seq_lens, parent.clone(), sizes.clone())
        for b in range(CFG.batch):
            n = int(sizes[b])
            err = np.abs(got[b, :n] - ref[b, :n])
            assert err.max() <= 2e-2 and err.mean() <= 2e-3
            assert np.all(got[b, n:] == 0.0)
        return got

    per_pass, parent, sizes, tokens = _grow(oracle, expand, attend, CFG.batch, V, greedy, CFG, seed=3)
    assert seen["expand_rows"] > 20 and int(sizes.min()) > 15
    # verification of the finished tree in one call: the rows every pass produced are still what it gives
    final = per_pass[-1][1]
    for n_then, rows in per_pass:
        for b in range(CFG.batch):
            n = int(n_then[b])
            assert np.abs(rows[b, :n] - final[b, :n]).max() <= 2e-2
