"""What the collectives must produce, written out as plain definitions.

Test infrastructure (see the package docstring).

* Reduce (Table 1; Section 3.4.2: every object is reduced once and only once): the target is
  the elementwise ``op`` over the selected objects.  For fp32 the bit pattern depends on the
  association, so :func:`tree_reduce` evaluates the final tree with each node combining its
  operands in the order of the placement traversal of Section 3.4.2 -- first child's result,
  the node's own object, then the remaining children's results, left to right:
  ``P_v = (((P_c1 op O_v) op P_c2) ... op P_cd)``; a leaf is its object, absent children are
  skipped.  bf16 inputs are widened to fp32 (exact) and reduced in fp32.
* :func:`naive_sum_f64` is the brute-force check: a left-to-right fp64 sum of the same objects.
* Broadcast: every receiver holds the source's bytes.
"""
from __future__ import annotations

import numpy as np

from .reduce_tree import children

OP_SUM, OP_MIN, OP_MAX = 0, 1, 2


def widen(a: np.ndarray) -> np.ndarray:
    """fp32 view of an object: float32 as is, bf16 bit patterns (uint16) widened exactly."""
    if a.dtype == np.float32:
        return a
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise TypeError(a.dtype)


def combine(a: np.ndarray, b: np.ndarray, op: int) -> np.ndarray:
    if op == OP_SUM:
        return np.add(a, b, dtype=np.float32)
    if op == OP_MIN:
        return np.where(b < a, b, a)
    if op == OP_MAX:
        return np.where(a < b, b, a)
    raise ValueError(op)


def tree_reduce(obj_at: list[int], d: int, objects: dict, op: int = OP_SUM, lo: int = 0, hi=None) -> np.ndarray:
    """Evaluate the tree whose position p holds object ``obj_at[p]`` over elements [lo, hi)."""
    k = len(obj_at)

    def own(p):
        return widen(objects[obj_at[p]][lo:hi])

    def result(p):
        ch = children(p, d, k)
        if not ch:
            return own(p)
        acc = combine(result(ch[0]), own(p), op)
        for c in ch[1:]:
            acc = combine(acc, result(c), op)
        return acc

    return np.array(result(0), dtype=np.float32, copy=True)


def naive_sum_f64(members: list[int], objects: dict, lo: int = 0, hi=None) -> np.ndarray:
    acc = np.zeros(len(widen(objects[members[0]][lo:hi])), dtype=np.float64)
    for m in members:
        acc = acc + widen(objects[m][lo:hi]).astype(np.float64)
    return acc


def naive_reduce_f32(members: list[int], objects: dict, op: int = OP_SUM) -> np.ndarray:
    """Left-to-right fp32 reduce in the given order (equals the chain and star trees)."""
    acc = widen(objects[members[0]]).copy()
    for m in members[1:]:
        acc = combine(acc, widen(objects[m]), op)
    return acc
