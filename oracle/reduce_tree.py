"""Reduce schedule: tree shape, arrival-order placement, k-of-m selection, failure edits.

Test infrastructure (see the package docstring).  Follows Section 3.4.2 and Section 3.5.2
of the paper; the figure that draws the tree did not survive, so the shape is the reading
that reproduces every statement of the text:

* the tree over ``k`` objects is the complete d-ary tree on positions ``0..k-1`` in level
  order (children of ``p`` are ``d*p+1 .. d*p+d`` where they exist).  ``d = 1`` is the chain,
  ``d >= k-1`` the star of Section 3.4.2, and the height is about ``log_d k`` (Eq. 1);
* arriving objects take positions in the generalised in-order traversal of Section 3.4.2:
  first child's subtree, the node itself, then the second ... d-th child's subtrees;
* construction stops once ``k`` objects are in the tree; later arrivals are spares;
* Section 3.5.2: a failed object's node leaves the tree at once and the next ready source
  takes its place; every ancestor clears what it had reduced.  Clearing is tracked per
  chunk: only chunk indices the departed object had delivered can have been merged.
* Build-defined (the paper blocks until a failed task is rebuilt): when fewer live sources
  remain than positions, the tree shrinks by its last level-order position; an object
  sitting there moves into the vacated position.
"""
from __future__ import annotations

from dataclasses import dataclass, field

EDIT_REPLACE = 1   # a spare took the vacated position immediately
EDIT_HOLE = 2      # the position stays open for the next arrival
EDIT_SHRINK = 3    # the tree lost its last position (an object there moved)


def children(p: int, d: int, k: int) -> list[int]:
    return [c for c in range(d * p + 1, d * p + d + 1) if c < k]


def parent(p: int, d: int) -> int:
    return -1 if p == 0 else (p - 1) // d


def ancestors(p: int, d: int) -> list[int]:
    """Strict ancestors of p, nearest first."""
    out = []
    while p > 0:
        p = (p - 1) // d
        out.append(p)
    return out


def choose_degree(n: int, size_bytes: float, latency: float, bandwidth: float) -> int:
    """Eq. 1 and Section 4: among d = 1, 2 and n, the degree with the smallest estimated reduce time
    ``T(1) = n L + S/B``, ``T(d) = L log_d n + d S/B``.  Ties go to the smaller degree."""
    import math
    if n <= 1:
        return 1
    t1 = n * latency + size_bytes / bandwidth
    t2 = latency * math.log2(n) + 2.0 * size_bytes / bandwidth
    tn = latency + n * size_bytes / bandwidth          # log_n n = 1
    best, d = t1, 1
    if t2 < best:
        best, d = t2, 2
    if tn < best:
        best, d = tn, n
    return d


def inorder(k: int, d: int) -> list[int]:
    """Positions of the complete d-ary tree on k nodes in generalised in-order."""
    out: list[int] = []
    if k <= 0:
        return out
    # explicit stack: (position, next child index to descend into, emitted?)
    stack = [(0, 0)]
    while stack:
        p, stage = stack.pop()
        ch = children(p, d, k)
        if stage == 0:
            stack.append((p, 1))
            if ch:
                stack.append((ch[0], 0))
        else:
            out.append(p)
            for c in reversed(ch[1:]):
                stack.append((c, 0))
    return out


@dataclass
class ReduceEdit:
    epoch: int
    kind: int
    pos: int                 # position vacated / filled (-1 if none)
    old_obj: int             # object that left (-1 if none)
    new_obj: int             # object now at ``pos`` (-1 if the position is open or gone)
    moved_from: int          # position the new object came from (-1 if it was not in the tree)
    hi_failed: int           # chunks the departed object had delivered
    hi_moved: int            # chunks the moved object had delivered (0 if nothing moved)
    cleared: list[int] = field(default_factory=list)   # positions whose partial results are cleared

    def words(self) -> list[int]:
        return [self.epoch, self.kind, self.pos, self.old_obj, self.new_obj, self.moved_from,
                self.hi_failed, self.hi_moved, len(self.cleared), *self.cleared]


class ReduceSchedule:
    """Online builder: feed it arrivals and failures in timeline order."""

    def __init__(self, src_ids: list[int], k: int, d: int):
        if not (1 <= k <= len(src_ids)) or d < 1:
            raise ValueError("need 1 <= k <= n and d >= 1")
        self.src = list(src_ids)
        self.k0 = k
        self.k = k
        self.d = d
        self.alive = {s: True for s in self.src}
        self.arrived: list[int] = []
        self.obj_at: list[int] = [-1] * k
        self.pos_of: dict[int, int] = {}
        self.spares: list[int] = []
        self.placements: list[tuple[int, int]] = []
        self.edits: list[ReduceEdit] = []
        self.epoch = 0

    # -- queries
    def live_count(self) -> int:
        return sum(1 for s in self.src if self.alive[s])

    def assigned_count(self) -> int:
        return sum(1 for o in self.obj_at if o >= 0)

    def full(self) -> bool:
        return self.k > 0 and self.assigned_count() == self.k

    def members(self) -> list[int]:
        return [o for o in self.obj_at if o >= 0]

    def _first_open(self) -> int:
        for p in inorder(self.k, self.d):
            if self.obj_at[p] < 0:
                return p
        return -1

    def _assign(self, obj: int, p: int) -> None:
        self.obj_at[p] = obj
        self.pos_of[obj] = p
        self.placements.append((obj, p))

    # -- events
    def on_arrival(self, obj: int) -> None:
        """The object's location was published for the first time (possibly still partial)."""
        if obj not in self.alive or not self.alive[obj] or obj in self.arrived:
            return
        self.arrived.append(obj)
        p = self._first_open()
        if p < 0:
            self.spares.append(obj)
        else:
            self._assign(obj, p)

    def on_rejoin(self, obj: int) -> None:
        """A failed source was reconstructed (Section 3.5): it is a future again and will count as a new
        arrival when it is put again ("R7 can also be the rejoined R2", Section 3.5.2).  A tree that has
        shrunk in the meantime does not grow back."""
        if obj in self.alive and not self.alive[obj]:
            self.alive[obj] = True
            if obj in self.arrived:
                self.arrived.remove(obj)

    def on_fail(self, obj: int, delivered_chunks: int, delivered_of=None) -> None:
        """``obj`` is lost.  ``delivered_chunks`` is its published chunk prefix; ``delivered_of(o)``
        gives the prefix of another object (needed when one has to move)."""
        if obj not in self.alive or not self.alive[obj]:
            return
        self.alive[obj] = False
        if obj in self.spares:
            self.spares.remove(obj)
        p = self.pos_of.pop(obj, -1)
        if p >= 0:
            self.obj_at[p] = -1
            self.epoch += 1
            if self.spares:
                s = self.spares.pop(0)
                self._assign(s, p)
                self.edits.append(ReduceEdit(self.epoch, EDIT_REPLACE, p, obj, s, -1, delivered_chunks, 0,
                                             ancestors(p, self.d)))
                return
            if self.live_count() >= self.k:
                self.edits.append(ReduceEdit(self.epoch, EDIT_HOLE, p, obj, -1, -1, delivered_chunks, 0,
                                             ancestors(p, self.d)))
                return
            self._shrink(p, obj, delivered_chunks, delivered_of)
        elif self.live_count() < self.k:
            self.epoch += 1
            self._shrink(-1, -1, 0, delivered_of)

    def _shrink(self, p: int, old_obj: int, hi_failed: int, delivered_of) -> None:
        q = self.k - 1
        moved = self.obj_at[q]
        cleared = ancestors(p, self.d) if p >= 0 else []
        self.k -= 1
        self.obj_at.pop()
        dest, hi_moved, moved_from = -1, 0, -1
        if q != p and moved >= 0:
            dest = p if p >= 0 else self._first_open()
            hi_moved = delivered_of(moved) if delivered_of else 0
            moved_from = q
            for a in ancestors(q, self.d):
                if a not in cleared:
                    cleared.append(a)
            self._assign(moved, dest)
            new_obj = moved
        else:
            new_obj = -1
            dest = p if (p >= 0 and p != q) else -1
        self.edits.append(ReduceEdit(self.epoch, EDIT_SHRINK, dest, old_obj, new_obj, moved_from,
                                     hi_failed, hi_moved, cleared))

    # -- serialisation (the word layout the library's schedule dump also produces)
    def words(self, target_id: int) -> list[int]:
        w = [0x48504C52, target_id, len(self.src), self.k0, self.k, self.d, len(self.placements)]
        for o, p in self.placements:
            w += [o, p]
        w += list(self.obj_at)
        w += [parent(p, self.d) for p in range(self.k)]
        w += [len(self.spares), *self.spares]
        w.append(len(self.edits))
        for e in self.edits:
            w += e.words()
        return w
