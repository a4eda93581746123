"""ctypes binding of ``libeagle_verify.so``: argument marshalling only.

Every function takes torch CUDA tensors (device memory and streams are torch's), checks dtypes and
shapes, fills the C descriptor and calls the C ABI declared in ``include/eagle_verify.h`` on the
current CUDA stream.  All arithmetic happens in the library's kernels.  There is no fallback: if the
shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libeagle_verify.so"
EXPORTS = ["eagle_tree_verify_attn_workspace", "eagle_tree_verify_attn", "eagle_tree_accept",
           "eagle_tree_build_mask", "eagle_status_string", "eagle_launch_count",
           "eagle_tree_verify_attn_static", "eagle_tree_verify_attn_static_capacity",
           "eagle_tree_verify_step_host", "eagle_tree_verify_step_host_arena", "eagle_tree_commit",
           "eagle_tree_accept_logits", "eagle_tree_expand", "eagle_tree_verify_attn_paged",
           "eagle_tree_commit_paged", "eagle_tree_verify_step_host_bytes", "eagle_tree_accept_cluster_width",
           "eagle_tree_verify_plan", "eagle_tree_verify_attn_planned", "eagle_tree_verify_attn_planned_paged",
           "eagle_tree_verify_plan_masks", "eagle_set_wait_limit_ns", "eagle_test_stall_kv_producer",
           "eagle_tree_verify_attn_fp8", "eagle_tree_verify_attn_planned_fp8", "eagle_tree_verify_attn_paged_fp8",
           "eagle_tree_verify_attn_planned_paged_fp8", "eagle_tree_accept_cluster_width_greedy"]
_lib = None


class EagleError(RuntimeError):
    pass


class AttnDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("max_tree", ctypes.c_int32), ("kv_capacity", ctypes.c_int32),
                ("tree_sizes", ctypes.c_void_p), ("sm_scale", ctypes.c_float), ("num_splits", ctypes.c_int32),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t), ("status", ctypes.c_void_p),
                ("ev_attn_begin", ctypes.c_void_p), ("ev_attn_end", ctypes.c_void_p), ("shared_tree", ctypes.c_int32)]


class PagedKV(ctypes.Structure):
    _fields_ = [("k_pages", ctypes.c_void_p), ("v_pages", ctypes.c_void_p), ("block_table", ctypes.c_void_p),
                ("num_pages", ctypes.c_int32), ("page_size", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32)]


class AcceptDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("max_tree", ctypes.c_int32), ("vocab", ctypes.c_int32),
                ("path_cap", ctypes.c_int32), ("tree_sizes", ctypes.c_void_p), ("greedy", ctypes.c_void_p),
                ("accept_len", ctypes.c_void_p), ("status", ctypes.c_void_p), ("shared_tree", ctypes.c_int32)]


class CommitDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("batch", "num_kv_heads", "head_dim", "kv_capacity", "max_tree", "path_cap",
                                              "feature_dim")] + [("status", ctypes.c_void_p)]


class ExpandDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("batch", "rows", "vocab", "max_children")] + [("greedy", ctypes.c_void_p),
                                                                                            ("status", ctypes.c_void_p)]


class HostStep(ctypes.Structure):
    _fields_ = ([(n, ctypes.c_int32) for n in ("batch", "num_q_heads", "num_kv_heads", "head_dim", "max_tree", "kv_capacity",
                                                "vocab", "path_cap")] + [("sm_scale", ctypes.c_float)] +
                [(n, ctypes.c_void_p) for n in ("q", "k_cache", "v_cache", "seq_lens", "tree_sizes", "tree_parent", "target_probs",
                                                "draft_probs", "draft_tokens", "uniforms", "greedy", "out", "accepted_path",
                                                "bonus_token", "accept_len", "status", "arena")] + [("arena_bytes", ctypes.c_size_t)])


def load():
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise EagleError(f"{LIB_PATH} is missing: build it with `python -m paper_2401_15077_b200.build` "
                             "(there is no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(str(LIB_PATH))
        vp, i32 = ctypes.c_void_p, ctypes.c_int32
        lib.eagle_tree_verify_attn_workspace.argtypes = [ctypes.POINTER(AttnDesc)]
        lib.eagle_tree_verify_attn_workspace.restype = ctypes.c_size_t
        lib.eagle_tree_verify_attn.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp, vp, vp]
        lib.eagle_tree_verify_attn.restype = ctypes.c_int
        lib.eagle_tree_verify_attn_static.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp, vp, vp]
        lib.eagle_tree_verify_attn_static.restype = ctypes.c_int
        lib.eagle_tree_verify_attn_static_capacity.restype = ctypes.c_size_t
        lib.eagle_tree_verify_attn_paged.argtypes = [ctypes.POINTER(AttnDesc), vp, ctypes.POINTER(PagedKV), vp, vp, vp, vp]
        lib.eagle_tree_verify_attn_paged.restype = ctypes.c_int
        lib.eagle_tree_verify_attn_fp8.argtypes = [ctypes.POINTER(AttnDesc)] + [vp] * 9
        lib.eagle_tree_verify_attn_fp8.restype = ctypes.c_int
        lib.eagle_tree_verify_attn_planned_fp8.argtypes = [ctypes.POINTER(AttnDesc)] + [vp] * 7
        lib.eagle_tree_verify_attn_planned_fp8.restype = ctypes.c_int
        lib.eagle_tree_verify_attn_paged_fp8.argtypes = [ctypes.POINTER(AttnDesc), vp, ctypes.POINTER(PagedKV)] + [vp] * 6
        lib.eagle_tree_verify_attn_paged_fp8.restype = ctypes.c_int
        lib.eagle_tree_verify_attn_planned_paged_fp8.argtypes = [ctypes.POINTER(AttnDesc), vp, ctypes.POINTER(PagedKV)] + [vp] * 4
        lib.eagle_tree_verify_attn_planned_paged_fp8.restype = ctypes.c_int
        lib.eagle_tree_verify_plan.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, ctypes.POINTER(PagedKV), vp]
        lib.eagle_tree_verify_plan.restype = ctypes.c_int
        lib.eagle_tree_verify_attn_planned.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp]
        lib.eagle_tree_verify_attn_planned.restype = ctypes.c_int
        lib.eagle_tree_verify_attn_planned_paged.argtypes = [ctypes.POINTER(AttnDesc), vp, ctypes.POINTER(PagedKV), vp, vp]
        lib.eagle_tree_verify_attn_planned_paged.restype = ctypes.c_int
        lib.eagle_tree_verify_plan_masks.argtypes = [ctypes.POINTER(AttnDesc)]
        lib.eagle_tree_verify_plan_masks.restype = ctypes.c_void_p
        lib.eagle_set_wait_limit_ns.argtypes = [ctypes.c_uint64]
        lib.eagle_set_wait_limit_ns.restype = None
        lib.eagle_test_stall_kv_producer.argtypes = [i32]
        lib.eagle_test_stall_kv_producer.restype = None
        lib.eagle_tree_verify_step_host.argtypes = [ctypes.POINTER(HostStep), vp]
        lib.eagle_tree_verify_step_host.restype = ctypes.c_int
        lib.eagle_tree_verify_step_host_arena.argtypes = [ctypes.POINTER(HostStep)]
        lib.eagle_tree_verify_step_host_arena.restype = ctypes.c_size_t
        lib.eagle_tree_verify_step_host_bytes.argtypes = [ctypes.POINTER(HostStep), ctypes.POINTER(ctypes.c_size_t),
                                                          ctypes.POINTER(ctypes.c_size_t)]
        lib.eagle_tree_verify_step_host_bytes.restype = ctypes.c_int
        lib.eagle_tree_accept.argtypes = [ctypes.POINTER(AcceptDesc), vp, vp, vp, vp, vp, vp, vp, vp]
        lib.eagle_tree_accept.restype = ctypes.c_int
        lib.eagle_tree_accept_cluster_width.argtypes = [i32, i32]
        lib.eagle_tree_accept_cluster_width.restype = ctypes.c_int
        lib.eagle_tree_accept_cluster_width_greedy.argtypes = [i32, i32]
        lib.eagle_tree_accept_cluster_width_greedy.restype = ctypes.c_int
        lib.eagle_tree_accept_logits.argtypes = [ctypes.POINTER(AcceptDesc), vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp]
        lib.eagle_tree_accept_logits.restype = ctypes.c_int
        lib.eagle_tree_expand.argtypes = [ctypes.POINTER(ExpandDesc), vp, vp, vp, vp, vp, vp]
        lib.eagle_tree_expand.restype = ctypes.c_int
        lib.eagle_tree_commit.argtypes = [ctypes.POINTER(CommitDesc), vp, vp, vp, vp, vp, vp, vp, vp]
        lib.eagle_tree_commit.restype = ctypes.c_int
        lib.eagle_tree_commit_paged.argtypes = [ctypes.POINTER(CommitDesc), ctypes.POINTER(PagedKV), vp, vp, vp, vp, vp, vp]
        lib.eagle_tree_commit_paged.restype = ctypes.c_int
        lib.eagle_tree_build_mask.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
        lib.eagle_tree_build_mask.restype = ctypes.c_int
        lib.eagle_status_string.argtypes = [ctypes.c_int]
        lib.eagle_status_string.restype = ctypes.c_char_p
        lib.eagle_launch_count.restype = ctypes.c_uint64
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load().eagle_status_string(int(code)).decode()


def launch_count() -> int:
    return int(load().eagle_launch_count())


def _check(rc: int, what: str):
    if rc != 0:
        raise EagleError(f"{what} failed: {rc} ({status_string(rc)})")


def _dev(t, dtype, name, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise EagleError(f"{name} is required")
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise EagleError(f"{name} must be a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _attn_desc(q, num_kv_heads, kv_capacity, tree_sizes, sm_scale, num_splits, workspace, status, events, shared_tree=False):
    B, T, Hq, D = q.shape
    d = AttnDesc(B, Hq, int(num_kv_heads), D, T, int(kv_capacity), _dev(tree_sizes, torch.int32, "tree_sizes", True), float(sm_scale),
                 int(num_splits), None, 0, _dev(status, torch.int32, "status", True), None, None, 1 if shared_tree else 0)
    if workspace is not None:
        d.workspace = workspace.data_ptr()
        d.workspace_bytes = workspace.numel() * workspace.element_size()
    if events is not None:
        d.ev_attn_begin, d.ev_attn_end = events[0].cuda_event, events[1].cuda_event
    return d


def _check_tree(tree_parent, tree_sizes, B, T, shared_tree):
    want = (T,) if shared_tree else (B, T)
    if tuple(tree_parent.shape) != want:
        raise EagleError(f"tree_parent must be {want}")
    if tree_sizes is not None and tree_sizes.numel() != (1 if shared_tree else B):
        raise EagleError("tree_sizes has the wrong length")


def eagle_tree_verify_attn_workspace(batch, num_q_heads, num_kv_heads, head_dim, max_tree, num_splits=0) -> int:
    d = AttnDesc(batch, num_q_heads, num_kv_heads, head_dim, max_tree, 0, None, 0.0, num_splits, None, 0, None, None, None)
    n = load().eagle_tree_verify_attn_workspace(ctypes.byref(d))
    if n == 0:
        raise EagleError("unsupported attention shape")
    return int(n)


def alloc_workspace(q, k_cache, num_splits=0) -> torch.Tensor:
    """Device scratch for ``eagle_tree_verify_attn`` (uint8, 256-byte aligned by the torch allocator)."""
    B, T, Hq, D = q.shape
    n = eagle_tree_verify_attn_workspace(B, Hq, k_cache.shape[1], D, T, num_splits)
    return torch.empty(n, dtype=torch.uint8, device=q.device)


def eagle_tree_verify_attn(q, k_cache, v_cache, seq_lens, tree_parent, out=None, *, tree_sizes=None, sm_scale=0.0,
                           num_splits=0, workspace=None, status=None, events=None, shared_tree=False):
    """Tree-masked attention.  q [B,T,Hq,D] bf16; k_cache/v_cache [B,Hkv,S,D] bf16; seq_lens [B] int32;
    tree_parent [B,T] int32 (or [T] with ``shared_tree``: one tree for every sequence, tree_sizes then [1] or None);
    returns out [B,T,Hq,D] bf16.  ``events``: optional pair of recorded-capable torch.cuda.Event(enable_timing=True)
    placed around the attention kernel alone."""
    lib = load()
    if q.dim() != 4 or k_cache.dim() != 4 or k_cache.shape != v_cache.shape:
        raise EagleError("bad tensor ranks / shapes")
    B, T, Hq, D = q.shape
    if k_cache.shape[0] != B or k_cache.shape[3] != D or tuple(seq_lens.shape) != (B,):
        raise EagleError("inconsistent shapes")
    _check_tree(tree_parent, tree_sizes, B, T, shared_tree)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = alloc_workspace(q, k_cache, num_splits)
    d = _attn_desc(q, k_cache.shape[1], k_cache.shape[2], tree_sizes, sm_scale, num_splits, workspace, status, events, shared_tree)
    rc = lib.eagle_tree_verify_attn(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), _dev(k_cache, torch.bfloat16, "k_cache"),
                                    _dev(v_cache, torch.bfloat16, "v_cache"), _dev(seq_lens, torch.int32, "seq_lens"),
                                    _dev(tree_parent, torch.int32, "tree_parent"), _dev(out, torch.bfloat16, "out"), _stream())
    _check(rc, "eagle_tree_verify_attn")
    return out


def eagle_tree_verify_attn_paged(q, k_pages, v_pages, block_table, seq_lens, tree_parent, out=None, *, tree_sizes=None,
                                 sm_scale=0.0, num_splits=0, workspace=None, status=None, events=None, shared_tree=False):
    """Tree-masked attention over a paged cache.  k_pages/v_pages [num_pages,Hkv,page_size,D] bf16; block_table
    [B,max_pages_per_seq] int32: slot j of sequence b is row j % page_size of page block_table[b, j // page_size].
    Everything else as for ``eagle_tree_verify_attn``."""
    lib = load()
    if q.dim() != 4 or k_pages.dim() != 4 or k_pages.shape != v_pages.shape or block_table.dim() != 2:
        raise EagleError("bad tensor ranks / shapes")
    B, T, Hq, D = q.shape
    P, Hkv, ps = k_pages.shape[0], k_pages.shape[1], k_pages.shape[2]
    if k_pages.shape[3] != D or block_table.shape[0] != B or tuple(seq_lens.shape) != (B,):
        raise EagleError("inconsistent shapes")
    _check_tree(tree_parent, tree_sizes, B, T, shared_tree)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = alloc_workspace(q, k_pages, num_splits)
    d = _attn_desc(q, Hkv, 0, tree_sizes, sm_scale, num_splits, workspace, status, events, shared_tree)
    pk = PagedKV(_dev(k_pages, torch.bfloat16, "k_pages"), _dev(v_pages, torch.bfloat16, "v_pages"),
                 _dev(block_table, torch.int32, "block_table"), P, ps, block_table.shape[1])
    rc = lib.eagle_tree_verify_attn_paged(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), ctypes.byref(pk),
                                          _dev(seq_lens, torch.int32, "seq_lens"), _dev(tree_parent, torch.int32, "tree_parent"),
                                          _dev(out, torch.bfloat16, "out"), _stream())
    _check(rc, "eagle_tree_verify_attn_paged")
    return out


def eagle_tree_verify_attn_fp8(q, k_codes, v_codes, k_scale, v_scale, seq_lens, tree_parent, out=None, *, tree_sizes=None,
                               sm_scale=0.0, num_splits=0, workspace=None, status=None, events=None, shared_tree=False):
    """Tree-masked attention over a cache stored as fp8 e4m3 codes: k_codes / v_codes uint8 [B,Hkv,S,D] (D = 128),
    k_scale / v_scale fp32 [B,Hkv].  Everything else as for ``eagle_tree_verify_attn``."""
    lib = load()
    if q.dim() != 4 or k_codes.dim() != 4 or k_codes.shape != v_codes.shape:
        raise EagleError("bad tensor ranks / shapes")
    B, T, Hq, D = q.shape
    Hkv = k_codes.shape[1]
    if k_codes.shape[0] != B or k_codes.shape[3] != D or tuple(seq_lens.shape) != (B,) or tuple(k_scale.shape) != (B, Hkv) or \
            tuple(v_scale.shape) != (B, Hkv):
        raise EagleError("inconsistent shapes")
    _check_tree(tree_parent, tree_sizes, B, T, shared_tree)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = alloc_workspace(q, k_codes, num_splits)
    d = _attn_desc(q, Hkv, k_codes.shape[2], tree_sizes, sm_scale, num_splits, workspace, status, events, shared_tree)
    rc = lib.eagle_tree_verify_attn_fp8(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), _dev(k_codes, torch.uint8, "k_codes"),
                                        _dev(v_codes, torch.uint8, "v_codes"), _dev(k_scale, torch.float32, "k_scale"),
                                        _dev(v_scale, torch.float32, "v_scale"), _dev(seq_lens, torch.int32, "seq_lens"),
                                        _dev(tree_parent, torch.int32, "tree_parent"), _dev(out, torch.bfloat16, "out"), _stream())
    _check(rc, "eagle_tree_verify_attn_fp8")
    return out


def eagle_tree_verify_attn_paged_fp8(q, k_pages, v_pages, k_scale, v_scale, block_table, seq_lens, tree_parent, out=None, *,
                                     tree_sizes=None, sm_scale=0.0, num_splits=0, workspace=None, status=None, events=None,
                                     shared_tree=False):
    """Tree-masked attention over a paged cache of fp8 e4m3 codes: k_pages / v_pages uint8 [num_pages,Hkv,page_size,D]
    (D = 128), k_scale / v_scale fp32 [B,Hkv], block_table [B,max_pages_per_seq] int32."""
    lib = load()
    if q.dim() != 4 or k_pages.dim() != 4 or k_pages.shape != v_pages.shape or block_table.dim() != 2:
        raise EagleError("bad tensor ranks / shapes")
    B, T, Hq, D = q.shape
    P, Hkv, ps = k_pages.shape[0], k_pages.shape[1], k_pages.shape[2]
    if k_pages.shape[3] != D or block_table.shape[0] != B or tuple(seq_lens.shape) != (B,) or tuple(k_scale.shape) != (B, Hkv) or \
            tuple(v_scale.shape) != (B, Hkv):
        raise EagleError("inconsistent shapes")
    _check_tree(tree_parent, tree_sizes, B, T, shared_tree)
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = alloc_workspace(q, k_pages, num_splits)
    d = _attn_desc(q, Hkv, 0, tree_sizes, sm_scale, num_splits, workspace, status, events, shared_tree)
    pk = PagedKV(_dev(k_pages, torch.uint8, "k_pages"), _dev(v_pages, torch.uint8, "v_pages"),
                 _dev(block_table, torch.int32, "block_table"), P, ps, block_table.shape[1])
    rc = lib.eagle_tree_verify_attn_paged_fp8(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), ctypes.byref(pk),
                                              _dev(k_scale, torch.float32, "k_scale"), _dev(v_scale, torch.float32, "v_scale"),
                                              _dev(seq_lens, torch.int32, "seq_lens"), _dev(tree_parent, torch.int32, "tree_parent"),
                                              _dev(out, torch.bfloat16, "out"), _stream())
    _check(rc, "eagle_tree_verify_attn_paged_fp8")
    return out


class VerifyPlan:
    """The plan of one verification pass (tree masks + work split), made once by ``eagle_tree_verify_plan`` and used by
    every layer's ``attend`` / ``attend_paged``.  Holds the descriptor fields and the workspace; marshalling only."""

    def __init__(self, shape, num_kv_heads, kv_capacity, tree_sizes, num_splits, workspace, shared_tree, paged):
        self.shape, self.num_kv_heads, self.kv_capacity = tuple(shape), int(num_kv_heads), int(kv_capacity)
        self.tree_sizes, self.num_splits, self.workspace = tree_sizes, int(num_splits), workspace
        self.shared_tree, self.paged = bool(shared_tree), paged

    def _desc(self, q_like_shape, sm_scale, status, events):
        B, T, Hq, D = q_like_shape
        d = AttnDesc(B, Hq, self.num_kv_heads, D, T, self.kv_capacity, _dev(self.tree_sizes, torch.int32, "tree_sizes", True),
                     float(sm_scale), self.num_splits, self.workspace.data_ptr(), self.workspace.numel(),
                     _dev(status, torch.int32, "status", True), None, None, 1 if self.shared_tree else 0)
        if events is not None:
            d.ev_attn_begin, d.ev_attn_end = events[0].cuda_event, events[1].cuda_event
        return d

    def masks(self):
        """Device address of the plan's ancestor masks (uint64 [B, T_max]) as an int64 tensor copy."""
        B, T = self.shape[0], self.shape[1]
        d = self._desc(self.shape, 0.0, None, None)
        ptr = load().eagle_tree_verify_plan_masks(ctypes.byref(d))
        if not ptr:
            raise EagleError("eagle_tree_verify_plan_masks failed")
        off = ptr - self.workspace.data_ptr()
        return self.workspace[off:off + B * T * 8].view(torch.int64).view(B, T).clone()

    def attend(self, q, k_cache, v_cache, out=None, *, sm_scale=0.0, status=None, events=None):
        if tuple(q.shape) != self.shape or k_cache.shape != v_cache.shape or k_cache.shape[2] != self.kv_capacity:
            raise EagleError("tensors do not match the plan")
        if out is None:
            out = torch.empty_like(q)
        d = self._desc(q.shape, sm_scale, status, events)
        rc = load().eagle_tree_verify_attn_planned(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), _dev(k_cache, torch.bfloat16, "k_cache"),
                                                   _dev(v_cache, torch.bfloat16, "v_cache"), _dev(out, torch.bfloat16, "out"), _stream())
        _check(rc, "eagle_tree_verify_attn_planned")
        return out

    def attend_fp8(self, q, k_codes, v_codes, k_scale, v_scale, out=None, *, sm_scale=0.0, status=None, events=None):
        if tuple(q.shape) != self.shape or k_codes.shape != v_codes.shape or k_codes.shape[2] != self.kv_capacity:
            raise EagleError("tensors do not match the plan")
        if out is None:
            out = torch.empty_like(q)
        d = self._desc(q.shape, sm_scale, status, events)
        rc = load().eagle_tree_verify_attn_planned_fp8(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), _dev(k_codes, torch.uint8, "k_codes"),
                                                       _dev(v_codes, torch.uint8, "v_codes"), _dev(k_scale, torch.float32, "k_scale"),
                                                       _dev(v_scale, torch.float32, "v_scale"), _dev(out, torch.bfloat16, "out"), _stream())
        _check(rc, "eagle_tree_verify_attn_planned_fp8")
        return out

    def attend_paged(self, q, k_pages, v_pages, block_table, out=None, *, sm_scale=0.0, status=None, events=None):
        if tuple(q.shape) != self.shape:
            raise EagleError("tensors do not match the plan")
        if out is None:
            out = torch.empty_like(q)
        d = self._desc(q.shape, sm_scale, status, events)
        pk = PagedKV(_dev(k_pages, torch.bfloat16, "k_pages"), _dev(v_pages, torch.bfloat16, "v_pages"),
                     _dev(block_table, torch.int32, "block_table"), k_pages.shape[0], k_pages.shape[2], block_table.shape[1])
        rc = load().eagle_tree_verify_attn_planned_paged(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), ctypes.byref(pk),
                                                         _dev(out, torch.bfloat16, "out"), _stream())
        _check(rc, "eagle_tree_verify_attn_planned_paged")
        return out

    def attend_paged_fp8(self, q, k_pages, v_pages, k_scale, v_scale, block_table, out=None, *, sm_scale=0.0, status=None, events=None):
        """One layer over a paged cache of fp8 codes, on a plan made with ``paged=``."""
        if tuple(q.shape) != self.shape:
            raise EagleError("tensors do not match the plan")
        if out is None:
            out = torch.empty_like(q)
        d = self._desc(q.shape, sm_scale, status, events)
        pk = PagedKV(_dev(k_pages, torch.uint8, "k_pages"), _dev(v_pages, torch.uint8, "v_pages"),
                     _dev(block_table, torch.int32, "block_table"), k_pages.shape[0], k_pages.shape[2], block_table.shape[1])
        rc = load().eagle_tree_verify_attn_planned_paged_fp8(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), ctypes.byref(pk),
                                                             _dev(k_scale, torch.float32, "k_scale"), _dev(v_scale, torch.float32, "v_scale"),
                                                             _dev(out, torch.bfloat16, "out"), _stream())
        _check(rc, "eagle_tree_verify_attn_planned_paged_fp8")
        return out


def eagle_tree_verify_plan(shape, num_kv_heads, kv_capacity, seq_lens, tree_parent, *, tree_sizes=None, num_splits=0,
                           workspace=None, status=None, shared_tree=False, paged=None) -> VerifyPlan:
    """Plans one verification pass: ``shape`` = (B, T_max, Hq, D) of q / out.  ``paged`` = (block_table, num_pages,
    page_size) for a paged cache (``kv_capacity`` is then ignored).  Returns the plan that ``attend`` takes."""
    B, T, Hq, D = shape
    _check_tree(tree_parent, tree_sizes, B, T, shared_tree)
    if workspace is None:
        n = eagle_tree_verify_attn_workspace(B, Hq, num_kv_heads, D, T, num_splits)
        workspace = torch.empty(n, dtype=torch.uint8, device=seq_lens.device)
    plan = VerifyPlan(shape, num_kv_heads, 0 if paged else kv_capacity, tree_sizes, num_splits, workspace, shared_tree, paged)
    d = plan._desc(shape, 0.0, status, None)
    pk = None
    if paged is not None:
        table, num_pages, page_size = paged
        pk = ctypes.byref(PagedKV(None, None, _dev(table, torch.int32, "block_table"), int(num_pages), int(page_size), table.shape[1]))
    rc = load().eagle_tree_verify_plan(ctypes.byref(d), _dev(seq_lens, torch.int32, "seq_lens"), _dev(tree_parent, torch.int32, "tree_parent"),
                                       pk, _stream())
    _check(rc, "eagle_tree_verify_plan")
    return plan


def set_wait_limit_ns(ns: int):
    load().eagle_set_wait_limit_ns(int(ns))


def test_stall_kv_producer(after_tiles: int):
    load().eagle_test_stall_kv_producer(int(after_tiles))


def eagle_tree_verify_attn_static(q, k_cache, v_cache, seq_lens, tree_parent, out, *, tree_sizes=None, sm_scale=0.0,
                                  num_splits=0, status=None, shared_tree=False):
    """Tree-masked attention for callers that may not allocate: same arguments and results as
    ``eagle_tree_verify_attn``, but no workspace is passed and none is allocated here either (the library's fixed
    device array is used; ``out`` must be given).  Raises if the shape needs more than that array holds."""
    lib = load()
    B, T, Hq, D = q.shape
    if k_cache.shape[0] != B or k_cache.shape[3] != D or tuple(seq_lens.shape) != (B,):
        raise EagleError("inconsistent shapes")
    _check_tree(tree_parent, tree_sizes, B, T, shared_tree)
    d = _attn_desc(q, k_cache.shape[1], k_cache.shape[2], tree_sizes, sm_scale, num_splits, None, status, None, shared_tree)
    rc = lib.eagle_tree_verify_attn_static(ctypes.byref(d), _dev(q, torch.bfloat16, "q"), _dev(k_cache, torch.bfloat16, "k_cache"),
                                           _dev(v_cache, torch.bfloat16, "v_cache"), _dev(seq_lens, torch.int32, "seq_lens"),
                                           _dev(tree_parent, torch.int32, "tree_parent"), _dev(out, torch.bfloat16, "out"), _stream())
    _check(rc, "eagle_tree_verify_attn_static")
    return out


def static_capacity() -> int:
    return int(load().eagle_tree_verify_attn_static_capacity())


def eagle_tree_accept(target_probs, draft_probs, draft_tokens, tree_parent, uniforms, accepted_path=None,
                      bonus_token=None, *, tree_sizes=None, greedy=None, accept_len=None, status=None, path_cap=None,
                      temperature=None, shared_tree=False):
    """Acceptance walk.  target_probs [B,T+1,V] fp32; draft_probs [B,T,V] fp32; draft_tokens/tree_parent [B,T]
    int32; uniforms [B,T+1] fp32.  Returns (accepted_path [B,path_cap] int32, bonus_token [B] int32).
    With ``temperature`` the two tensors hold logits (``eagle_tree_accept_logits``)."""
    lib = load()
    B, T1, V = target_probs.shape
    T = T1 - 1
    dev = target_probs.device
    cap = T if path_cap is None else int(path_cap)
    if accepted_path is None:
        accepted_path = torch.empty((B, cap), dtype=torch.int32, device=dev)
    if bonus_token is None:
        bonus_token = torch.empty((B,), dtype=torch.int32, device=dev)
    if tuple(draft_tokens.shape) != (B, T) or tuple(accepted_path.shape) != (B, cap):
        raise EagleError("inconsistent shapes")
    _check_tree(tree_parent, tree_sizes, B, T, shared_tree)
    if draft_probs is not None and tuple(draft_probs.shape) != (B, T, V):
        raise EagleError("draft_probs must be [B, T, V]")
    if uniforms is not None and tuple(uniforms.shape) != (B, T + 1):
        raise EagleError("uniforms must be [B, T+1]")
    d = AcceptDesc(B, T, V, cap, _dev(tree_sizes, torch.int32, "tree_sizes", True), _dev(greedy, torch.uint8, "greedy", True),
                   _dev(accept_len, torch.int32, "accept_len", True), _dev(status, torch.int32, "status", True),
                   1 if shared_tree else 0)
    head = (ctypes.byref(d), _dev(target_probs, torch.float32, "target_probs"), _dev(draft_probs, torch.float32, "draft_probs", True),
            _dev(draft_tokens, torch.int32, "draft_tokens"), _dev(tree_parent, torch.int32, "tree_parent"),
            _dev(uniforms, torch.float32, "uniforms", True))
    tail = (_dev(accepted_path, torch.int32, "accepted_path"), _dev(bonus_token, torch.int32, "bonus_token"), _stream())
    if temperature is None:
        _check(lib.eagle_tree_accept(*head, *tail), "eagle_tree_accept")
    else:
        _check(lib.eagle_tree_accept_logits(*head, float(temperature), *tail), "eagle_tree_accept_logits")
    return accepted_path, bonus_token


def eagle_tree_accept_cluster_width(batch: int, vocab: int, all_greedy: bool = False) -> int:
    """0 when a warp walks each tree, else the CTAs per cluster (1, 2, 4, 8) an acceptance call of this size uses here
    (``all_greedy``: a call without draft rows or uniforms)."""
    fn = load().eagle_tree_accept_cluster_width_greedy if all_greedy else load().eagle_tree_accept_cluster_width
    rc = fn(int(batch), int(vocab))
    if rc < 0:
        _check(rc, "eagle_tree_accept_cluster_width")
    return rc


def eagle_tree_accept_logits(target_logits, draft_logits, draft_tokens, tree_parent, uniforms, temperature, accepted_path=None,
                             bonus_token=None, **kw):
    """Acceptance walk on logits: rows are softmax(logits / temperature), never materialised."""
    return eagle_tree_accept(target_logits, draft_logits, draft_tokens, tree_parent, uniforms, accepted_path, bonus_token,
                             temperature=temperature, **kw)


def eagle_tree_build_mask(tree_parent, tree_sizes=None, status=None, with_depth=True):
    """Ancestor-or-self bit masks (int64 tensor holding the uint64 bit pattern) and depths (uint8)."""
    lib = load()
    B, T = tree_parent.shape
    anc = torch.empty((B, T), dtype=torch.int64, device=tree_parent.device)
    depth = torch.empty((B, T), dtype=torch.uint8, device=tree_parent.device) if with_depth else None
    rc = lib.eagle_tree_build_mask(_dev(tree_parent, torch.int32, "tree_parent"), _dev(tree_sizes, torch.int32, "tree_sizes", True),
                                   B, T, anc.data_ptr(), None if depth is None else depth.data_ptr(),
                                   _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "eagle_tree_build_mask")
    return anc, depth


def eagle_tree_expand(draft_probs, num_children, max_children, uniforms=None, greedy=None, status=None, with_probs=True):
    """Child tokens of draft-tree nodes: top-k per row for greedy sequences, k inverse-CDF draws otherwise.
    draft_probs [B, R, V] fp32, num_children [B, R] int32, uniforms [B, R, K] fp32.  Returns (tokens, probs) [B, R, K]."""
    lib = load()
    B, R, V = draft_probs.shape
    K = int(max_children)
    tokens = torch.empty((B, R, K), dtype=torch.int32, device=draft_probs.device)
    probs = torch.empty((B, R, K), dtype=torch.float32, device=draft_probs.device) if with_probs else None
    d = ExpandDesc(B, R, V, K, _dev(greedy, torch.uint8, "greedy", True), _dev(status, torch.int32, "status", True))
    rc = lib.eagle_tree_expand(ctypes.byref(d), _dev(draft_probs, torch.float32, "draft_probs"),
                               _dev(num_children, torch.int32, "num_children"), _dev(uniforms, torch.float32, "uniforms", True),
                               tokens.data_ptr(), None if probs is None else probs.data_ptr(), _stream())
    _check(rc, "eagle_tree_expand")
    return tokens, probs


def eagle_tree_commit(k_cache, v_cache, seq_lens, accepted_path, max_tree, features=None, features_out=None,
                      new_seq_lens=None, status=None):
    """Commit of the accepted path: moves the accepted nodes' K/V rows into the next prefix slots IN PLACE and gathers
    their feature vectors.  Returns (new_seq_lens, features_out); both are allocated when not passed in."""
    lib = load()
    B, Hkv, S, D = k_cache.shape
    cap = accepted_path.shape[1]
    F = 0 if features is None else features.shape[2]
    if new_seq_lens is None:
        new_seq_lens = torch.empty((B,), dtype=torch.int32, device=k_cache.device)
    if features is not None and features_out is None:
        features_out = torch.empty((B, cap, F), dtype=torch.bfloat16, device=k_cache.device)
    d = CommitDesc(B, Hkv, D, S, max_tree, cap, F, _dev(status, torch.int32, "status", True))
    rc = lib.eagle_tree_commit(ctypes.byref(d), _dev(k_cache, torch.bfloat16, "k_cache"), _dev(v_cache, torch.bfloat16, "v_cache", True),
                               _dev(seq_lens, torch.int32, "seq_lens"), _dev(accepted_path, torch.int32, "accepted_path"),
                               _dev(features, torch.bfloat16, "features", True), _dev(features_out, torch.bfloat16, "features_out", True),
                               _dev(new_seq_lens, torch.int32, "new_seq_lens"), _stream())
    _check(rc, "eagle_tree_commit")
    return new_seq_lens, features_out


def eagle_tree_commit_paged(k_pages, v_pages, block_table, seq_lens, accepted_path, max_tree, features=None, features_out=None,
                            new_seq_lens=None, status=None):
    """``eagle_tree_commit`` on a paged cache: k_pages / v_pages [num_pages, Hkv, page_size, D] are updated IN PLACE through
    block_table [B, max_pages_per_seq].  Returns (new_seq_lens, features_out)."""
    lib = load()
    P, Hkv, ps, D = k_pages.shape
    B = seq_lens.shape[0]
    cap = accepted_path.shape[1]
    F = 0 if features is None else features.shape[2]
    if new_seq_lens is None:
        new_seq_lens = torch.empty((B,), dtype=torch.int32, device=k_pages.device)
    if features is not None and features_out is None:
        features_out = torch.empty((B, cap, F), dtype=torch.bfloat16, device=k_pages.device)
    d = CommitDesc(B, Hkv, D, 0, max_tree, cap, F, _dev(status, torch.int32, "status", True))
    pk = PagedKV(_dev(k_pages, torch.bfloat16, "k_pages"), _dev(v_pages, torch.bfloat16, "v_pages", True),
                 _dev(block_table, torch.int32, "block_table"), P, ps, block_table.shape[1])
    rc = lib.eagle_tree_commit_paged(ctypes.byref(d), ctypes.byref(pk), _dev(seq_lens, torch.int32, "seq_lens"),
                                     _dev(accepted_path, torch.int32, "accepted_path"), _dev(features, torch.bfloat16, "features", True),
                                     _dev(features_out, torch.bfloat16, "features_out", True),
                                     _dev(new_seq_lens, torch.int32, "new_seq_lens"), _stream())
    _check(rc, "eagle_tree_commit_paged")
    return new_seq_lens, features_out


class HostStepRunner:
    """One verification step from (pinned) host tensors through ``eagle_tree_verify_step_host``.

    ``host`` maps q, k_cache, v_cache, seq_lens, tree_sizes, tree_parent, target_probs, draft_probs, draft_tokens,
    uniforms, greedy to CPU tensors; outputs land in the pinned tensors ``out``, ``accepted_path``, ``bonus_token``,
    ``accept_len``, ``status`` of this object once the stream has drained.  The device arena is allocated once here."""

    def __init__(self, host: dict, device):
        lib = load()
        self.host = host
        q, k, tp = host["q"], host["k_cache"], host["target_probs"]
        B, T, Hq, D = q.shape
        self.out = torch.empty(q.shape, dtype=q.dtype).pin_memory()
        self.accepted_path = torch.empty((B, T), dtype=torch.int32).pin_memory()
        self.bonus_token = torch.empty((B,), dtype=torch.int32).pin_memory()
        self.accept_len = torch.empty((B,), dtype=torch.int32).pin_memory()
        self.status = torch.zeros((1,), dtype=torch.int32).pin_memory()
        s = HostStep()
        s.batch, s.num_q_heads, s.num_kv_heads, s.head_dim, s.max_tree = B, Hq, k.shape[1], D, T
        s.kv_capacity, s.vocab, s.path_cap, s.sm_scale = k.shape[2], tp.shape[2], T, 0.0
        for name in ("q", "k_cache", "v_cache", "seq_lens", "tree_sizes", "tree_parent", "target_probs", "draft_probs",
                     "draft_tokens", "uniforms", "greedy"):
            t = host.get(name)
            setattr(s, name, None if t is None else t.data_ptr())
        s.out, s.accepted_path, s.bonus_token = self.out.data_ptr(), self.accepted_path.data_ptr(), self.bonus_token.data_ptr()
        s.accept_len, s.status = self.accept_len.data_ptr(), self.status.data_ptr()
        n = lib.eagle_tree_verify_step_host_arena(ctypes.byref(s))
        if n == 0:
            raise EagleError("unsupported shape for the host step")
        self.arena = torch.empty(n, dtype=torch.uint8, device=device)
        s.arena, s.arena_bytes = self.arena.data_ptr(), n
        self.step = s
        # what the call copies: whole tensors, or (when that saves enough) only the visible cache slots and existing rows
        self.full_h2d_bytes = sum(t.numel() * t.element_size() for t in host.values() if t is not None)
        h2d, d2h = ctypes.c_size_t(0), ctypes.c_size_t(0)
        _check(lib.eagle_tree_verify_step_host_bytes(ctypes.byref(s), ctypes.byref(h2d), ctypes.byref(d2h)),
               "eagle_tree_verify_step_host_bytes")
        self.h2d_bytes, self.d2h_bytes = int(h2d.value), int(d2h.value)

    def run(self):
        _check(load().eagle_tree_verify_step_host(ctypes.byref(self.step), _stream()), "eagle_tree_verify_step_host")
