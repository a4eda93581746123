"""Seeded synthetic inputs for the tree-verification step.

This module holds no arithmetic of the method itself (no masking, attention or acceptance rule):
it only draws inputs.  Both the CUDA tests/bench and the CPU oracle's tests take their inputs from
here, so the two sides see identical data.  Everything is generated on the CPU with
``torch.Generator`` seeds ``15077*1000 + 100*config_index + stream``.

The shapes stand in for the models the paper evaluates (Vicuna/LLaMA2-Chat 7B..70B, Mixtral 8x7B;
Sec. 4): the paper's prompts and its fixed draft tree are not available, so random trees with a
depth limit and a branching cap are used, and logits are Gaussian.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

STREAMS = dict(q=0, k=1, v=2, tree=3, target=4, draft=5, tokens=6, uniforms=7, lens=8, sizes=9, paths=10, features=11, pages=12)


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    index: int
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    prefix: tuple          # (lo, hi) inclusive range of committed prefix lengths
    tree: tuple            # (lo, hi) inclusive range of tree sizes
    max_depth: int
    child_cap: int         # 0 = no cap
    vocab: int
    greedy: str            # "none" | "all" | "half"

    @property
    def max_tree(self) -> int:
        return self.tree[1]


CONFIGS = {
    c.name: c
    for c in [
        VerifyConfig("tiny", 0, 1, 8, 8, 64, (256, 256), (8, 8), 4, 0, 1000, "none"),
        VerifyConfig("7b_mha", 1, 1, 32, 32, 128, (2048, 2048), (26, 26), 5, 0, 32000, "none"),
        VerifyConfig("70b_gqa", 2, 4, 64, 8, 128, (4096, 4096), (60, 60), 6, 10, 32000, "none"),
        VerifyConfig("mixtral_gqa", 3, 8, 32, 8, 128, (16384, 16384), (26, 26), 5, 0, 32000, "none"),
        VerifyConfig("serving_mix", 4, 64, 32, 8, 128, (512, 8192), (16, 64), 6, 0, 32000, "half"),
    ]
}


def seed_for(cfg_index: int, stream: str, salt: int = 0) -> int:
    return 15077 * 1000 + 100 * cfg_index + STREAMS[stream] + 1000003 * salt


def _gen(cfg_index: int, stream: str, salt: int = 0) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed_for(cfg_index, stream, salt))
    return g


def random_tree(size: int, max_depth: int, child_cap: int, gen: torch.Generator) -> list:
    """parent[i] uniform over the admissible earlier nodes (and -1 = the context): those whose depth is
    below ``max_depth`` and that have fewer than ``child_cap`` children (0 = no cap)."""
    parent, depth, kids = [], [], {}
    for i in range(size):
        ok = [c for c in range(-1, i)
              if (0 if c < 0 else depth[c]) < max_depth and (child_cap <= 0 or kids.get(c, 0) < child_cap)]
        c = ok[int(torch.randint(len(ok), (1,), generator=gen))]
        parent.append(c)
        depth.append(1 if c < 0 else depth[c] + 1)
        kids[c] = kids.get(c, 0) + 1
    return parent


@dataclass
class AttnInputs:
    cfg: VerifyConfig
    q: torch.Tensor            # bf16 [B, T_max, Hq, D]
    k_cache: torch.Tensor      # bf16 [B, Hkv, S_cap, D]
    v_cache: torch.Tensor
    seq_lens: torch.Tensor     # int32 [B]
    tree_sizes: torch.Tensor   # int32 [B]
    tree_parent: torch.Tensor  # int32 [B, T_max]
    kv_capacity: int = 0
    extra: dict = field(default_factory=dict)

    def algorithmic_bytes(self) -> int:
        """K and V rows of every visible slot plus Q and O rows: what the step has to move."""
        c = self.cfg
        kv = int((self.seq_lens.long() + self.tree_sizes.long()).sum()) * c.num_kv_heads * c.head_dim * 2 * 2
        qo = int(self.tree_sizes.long().sum()) * c.num_q_heads * c.head_dim * 2 * 2
        return kv + qo

    def algorithmic_flops(self) -> int:
        c = self.cfg
        keys = self.seq_lens.long() + self.tree_sizes.long()
        return int((keys * self.tree_sizes.long()).sum()) * c.num_q_heads * c.head_dim * 4


def make_trees(cfg: VerifyConfig, salt: int = 0):
    gs, gt = _gen(cfg.index, "sizes", salt), _gen(cfg.index, "tree", salt)
    B, T = cfg.batch, cfg.max_tree
    sizes = torch.randint(cfg.tree[0], cfg.tree[1] + 1, (B,), generator=gs, dtype=torch.int32)
    parent = torch.full((B, T), -1, dtype=torch.int32)
    for b in range(B):
        n = int(sizes[b])
        parent[b, :n] = torch.tensor(random_tree(n, cfg.max_depth, cfg.child_cap, gt), dtype=torch.int32)
        # padding entries are never read; give them values that would be invalid if they were
        parent[b, n:] = 2 ** 30
    return sizes, parent


def make_attn_inputs(cfg: VerifyConfig, salt: int = 0, poison: bool = True, capacity_pad: int = 0) -> AttnInputs:
    """Q/K/V ~ N(0,1) rounded to bf16; cache slots past prefix+tree hold NaN when ``poison``."""
    B, T, Hq, Hkv, D = cfg.batch, cfg.max_tree, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
    gl = _gen(cfg.index, "lens", salt)
    lens = torch.randint(cfg.prefix[0], cfg.prefix[1] + 1, (B,), generator=gl, dtype=torch.int32)
    sizes, parent = make_trees(cfg, salt)
    cap = int((lens + sizes).max()) + capacity_pad
    gq, gk, gv = _gen(cfg.index, "q", salt), _gen(cfg.index, "k", salt), _gen(cfg.index, "v", salt)
    q = torch.randn((B, T, Hq, D), generator=gq, dtype=torch.float32).to(torch.bfloat16)
    fill = float("nan") if poison else 0.0
    k = torch.full((B, Hkv, cap, D), fill, dtype=torch.bfloat16)
    v = torch.full((B, Hkv, cap, D), fill, dtype=torch.bfloat16)
    for b in range(B):
        n = int(lens[b] + sizes[b])
        k[b, :, :n] = torch.randn((Hkv, n, D), generator=gk, dtype=torch.float32).to(torch.bfloat16)
        v[b, :, :n] = torch.randn((Hkv, n, D), generator=gv, dtype=torch.float32).to(torch.bfloat16)
        if poison:
            q[b, int(sizes[b]):] = float("nan")
    return AttnInputs(cfg, q, k, v, lens, sizes, parent, cap)


@dataclass
class PagedKV:
    k_pages: torch.Tensor      # bf16 [num_pages, Hkv, page_size, D]
    v_pages: torch.Tensor
    block_table: torch.Tensor  # int32 [B, max_pages_per_seq]
    page_size: int


def make_paged_cache(inp: AttnInputs, page_size: int, salt: int = 0, spare_pages: int = 3, poison: bool = True, codes=None) -> PagedKV:
    """The same keys and values as ``inp`` stored in pages of ``page_size`` slots, scattered over the pool by a seeded
    permutation.  Only pages that hold a visible slot get a table entry; the other entries are -1, and rows of slots
    that are not visible (as well as ``spare_pages`` unused pages) hold NaN when ``poison``.  With ``codes`` (an
    ``Fp8KV`` of the same cache) the pages hold its fp8 codes instead (uint8; the NaN code where not visible)."""
    cfg = inp.cfg
    B, Hkv, D = cfg.batch, cfg.num_kv_heads, cfg.head_dim
    vis = [int(inp.seq_lens[b] + inp.tree_sizes[b]) if int(inp.tree_sizes[b]) > 0 else 0 for b in range(B)]
    need = [(n + page_size - 1) // page_size for n in vis]
    max_pages = max(1, (inp.kv_capacity + page_size - 1) // page_size)
    total = sum(need) + spare_pages
    order = torch.randperm(total, generator=_gen(cfg.index, "pages", salt)).tolist()
    if codes is None:
        src_k, src_v = inp.k_cache, inp.v_cache
        fill, dtype = (float("nan") if poison else 0.0), torch.bfloat16
    else:
        src_k, src_v = codes.k_codes, codes.v_codes
        fill, dtype = (0x7F if poison else 0), torch.uint8
    kp = torch.full((max(total, 1), Hkv, page_size, D), fill, dtype=dtype)
    vp = torch.full((max(total, 1), Hkv, page_size, D), fill, dtype=dtype)
    table = torch.full((B, max_pages), -1, dtype=torch.int32)
    nxt = 0
    for b in range(B):
        for i in range(need[b]):
            page = order[nxt]
            nxt += 1
            table[b, i] = page
            rows = min(page_size, vis[b] - i * page_size)
            kp[page, :, :rows] = src_k[b, :, i * page_size:i * page_size + rows]
            vp[page, :, :rows] = src_v[b, :, i * page_size:i * page_size + rows]
    return PagedKV(kp, vp, table, page_size)


@dataclass
class Fp8KV:
    k_codes: torch.Tensor      # uint8 [B, Hkv, S_cap, D]: fp8 e4m3 codes
    v_codes: torch.Tensor
    k_scale: torch.Tensor      # fp32 [B, Hkv]
    v_scale: torch.Tensor


def make_fp8_cache(inp: AttnInputs, poison: bool = True, power_of_two_scales: bool = False) -> Fp8KV:
    """The keys and values of ``inp`` as a serving engine would store them in fp8: per (sequence, KV head) a scale
    amax / 448 over the visible slots and the codes of round(x / scale) to e4m3 (the library's conversion; this is input
    preparation, not part of the verification step).  Slots that are not visible hold the NaN code when ``poison``."""
    cfg = inp.cfg
    B, Hkv = cfg.batch, cfg.num_kv_heads
    out = []
    for x in (inp.k_cache, inp.v_cache):
        codes = torch.full(x.shape, 0x7F if poison else 0, dtype=torch.uint8)
        scale = torch.ones((B, Hkv), dtype=torch.float32)
        for b in range(B):
            n = int(inp.seq_lens[b] + inp.tree_sizes[b])
            if n == 0:
                continue
            vis = x[b, :, :n].float()
            s = vis.abs().amax(dim=(1, 2)).clamp_min(1e-12) / 448.0
            if power_of_two_scales:
                s = torch.exp2(torch.ceil(torch.log2(s)))
            scale[b] = s
            codes[b, :, :n] = (vis / s[:, None, None]).to(torch.float8_e4m3fn).view(torch.uint8)
        out += [codes, scale]
    return Fp8KV(out[0], out[2], out[1], out[3])


@dataclass
class AcceptInputs:
    cfg: VerifyConfig
    target_probs: torch.Tensor   # fp32 [B, T_max+1, V]
    draft_probs: torch.Tensor    # fp32 [B, T_max, V]
    draft_tokens: torch.Tensor   # int32 [B, T_max]
    tree_parent: torch.Tensor    # int32 [B, T_max]
    tree_sizes: torch.Tensor     # int32 [B]
    uniforms: torch.Tensor       # fp32 [B, T_max+1]
    greedy: torch.Tensor         # uint8 [B]


def make_accept_inputs(cfg: VerifyConfig, salt: int = 0, rho: float = 0.9, rho_greedy: float = 0.98,
                       trees=None, vocab: int | None = None, greedy: str | None = None, logits: bool = False) -> AcceptInputs:
    """Target logits ~ N(0, variance 2); draft logits = rho*target + sqrt(1-rho^2)*fresh (same marginal).
    Row i of ``draft_probs`` is the softmax of the draft logits at node i's parent; stochastic sequences
    draw node tokens i.i.d. from that row, greedy sequences give the j-th child the parent's rank-j draft
    token.  ``rho`` = 0 is the uncorrelated (rejection-heavy) case.  With ``logits`` the two tensors hold the logits
    themselves (for the entry point that takes logits); tokens are drawn the same way."""
    B, T = cfg.batch, cfg.max_tree
    V = vocab or cfg.vocab
    sizes, parent = trees if trees is not None else make_trees(cfg, salt)
    mode = greedy or cfg.greedy
    gflag = torch.zeros(B, dtype=torch.uint8)
    if mode == "all":
        gflag[:] = 1
    elif mode == "half":
        gflag[1::2] = 1
    gt, gd, gk, gu = (_gen(cfg.index, s, salt) for s in ("target", "draft", "tokens", "uniforms"))
    sigma = math.sqrt(2.0)
    target = torch.empty((B, T + 1, V), dtype=torch.float32)
    draft = torch.zeros((B, T, V), dtype=torch.float32)
    tokens = torch.zeros((B, T), dtype=torch.int32)
    for b in range(B):
        n = int(sizes[b])
        r = rho_greedy if gflag[b] else rho
        tl = torch.randn((T + 1, V), generator=gt, dtype=torch.float32) * sigma
        fresh = torch.randn((T + 1, V), generator=gd, dtype=torch.float32) * sigma
        dl = r * tl + math.sqrt(max(0.0, 1.0 - r * r)) * fresh
        target[b] = tl if logits else torch.softmax(tl, dim=-1)
        dprob = torch.softmax(dl, dim=-1)          # row c+1 = draft distribution after node c
        child_rank = {}
        for i in range(n):
            c = int(parent[b, i])
            draft[b, i] = dl[c + 1] if logits else dprob[c + 1]
            if gflag[b]:
                j = child_rank.get(c, 0)
                child_rank[c] = j + 1
                tokens[b, i] = int(torch.topk(dprob[c + 1], j + 1).indices[j])
            else:
                tokens[b, i] = int(torch.multinomial(dprob[c + 1], 1, generator=gk))
    uniforms = torch.rand((B, T + 1), generator=gu, dtype=torch.float32)
    return AcceptInputs(cfg, target, draft, tokens, parent, sizes, uniforms, gflag)


def make_accepted_paths(sizes: torch.Tensor, parent: torch.Tensor, path_cap: int, cfg_index: int, salt: int = 0) -> torch.Tensor:
    """One random chain per tree from a top-level node downwards (what an acceptance walk can return): at every node
    stop with probability 1/4, else move to a random child.  int32 [B, path_cap], -1 padded; an empty tree or an
    immediate stop gives an empty path."""
    g = _gen(cfg_index, "paths", salt)
    B, T = parent.shape
    out = torch.full((B, path_cap), -1, dtype=torch.int32)
    for b in range(B):
        n, cur, j = int(sizes[b]), -1, 0
        while j < path_cap:
            kids = [i for i in range(n) if int(parent[b, i]) == cur]
            if not kids or float(torch.rand((), generator=g)) < 0.25:
                break
            cur = kids[int(torch.randint(len(kids), (), generator=g))]
            out[b, j] = cur
            j += 1
    return out


def scaled(cfg: VerifyConfig, **kw) -> VerifyConfig:
    """A copy of ``cfg`` with some fields replaced (used for reduced-size parity cases)."""
    d = {f: getattr(cfg, f) for f in cfg.__dataclass_fields__}
    d.update(kw)
    return VerifyConfig(**d)
