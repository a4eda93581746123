"""Comparison of an acceptance result with the oracle's, decision by decision (test infrastructure, like the oracle:
used by the parity tests, the smoke check and the bench's parity record; holds none of the method's arithmetic).

With fixed uniforms the walk has one correct result; a floating-point decision that sits within rounding of its
boundary may still fall either way.  The stated rule: results must be identical, except that a difference is tolerated
when the oracle's margin AT THE FIRST DECISION THAT DIFFERS is below 1e-5 (everything after that decision follows
from it and proves nothing more).  The oracle returns its decisions in order (kind, node, margin); the other side's
decisions are recovered from its outputs, which is possible because both sides take the same decisions in the same
order until the first one that differs.
"""
import numpy as np

DEC_ACCEPT, DEC_REJECT, DEC_BONUS, DEC_ARGMAX = 0, 1, 2, 3


def first_differing_decision(ref, b, path, bonus, parent=None, tokens=None):
    """Index (into the oracle's decision list of sequence ``b``) of the first decision whose outcome the outputs
    ``path`` (row of accepted_path, -1 padded) and ``bonus`` contradict; None when they contradict none.

    ``parent`` / ``tokens`` (rows of tree_parent / draft_tokens) are needed for greedy sequences only, where a decision
    is an argmax and its outcome shows as the child moved to (the lowest-index child carrying that token) or as the
    emitted token."""
    n_dec = int(ref["n_dec"][b])
    rpath, rbonus = ref["accepted_path"][b], int(ref["bonus_token"][b])
    cap = len(rpath)
    depth = 0                         # accepted nodes so far (the two walks agree on them up to here)
    for d in range(n_dec):
        kind, node = int(ref["dec_kind"][b, d]), int(ref["dec_node"][b, d])
        mine = int(path[depth]) if depth < cap else -1   # what the other side did at this depth (-1: it stopped here)
        if kind == DEC_ACCEPT:
            if mine != node:
                return d
            depth += 1
        elif kind == DEC_REJECT:
            if mine == node:
                return d
        elif kind == DEC_BONUS:
            if mine != -1 or int(bonus) != rbonus:
                return d
        elif kind == DEC_ARGMAX:
            theirs = int(rpath[depth]) if depth < cap and depth < int(ref["accept_len"][b]) else -1
            if mine != theirs or (theirs == -1 and int(bonus) != rbonus):
                return d
            if theirs == -1:
                break
            depth += 1
        else:
            raise AssertionError(f"unknown decision kind {kind}")
    return None


def compare_with_oracle(ref, path, bonus, alen, greedy, margin=1e-5):
    """Asserts that (path, bonus, alen) equal the oracle's result ``ref`` for every sequence, tolerating a sequence only
    when the oracle's margin at the first differing decision is below ``margin`` and the sequence is not greedy.
    Returns the number of tolerated sequences."""
    same = (path == ref["accepted_path"]).all(axis=1) & (bonus == ref["bonus_token"]) & (alen == ref["accept_len"])
    tolerated = 0
    for b in np.nonzero(~same)[0]:
        assert greedy is None or not greedy[b], f"greedy sequence {b} differs"
        d = first_differing_decision(ref, b, path[b], bonus[b])
        assert d is not None, (b, "outputs differ but no decision does", path[b], ref["accepted_path"][b], alen[b], ref["accept_len"][b])
        m = float(ref["dec_margin"][b, d])
        assert m < margin, (b, d, int(ref["dec_kind"][b, d]), int(ref["dec_node"][b, d]), m, path[b], ref["accepted_path"][b],
                            bonus[b], ref["bonus_token"][b])
        tolerated += 1
    return tolerated
