"""Broadcast schedule: receiver-driven tree formation in virtual time, and failover.

Test infrastructure (see the package docstring).  Follows Section 3.4.1 and Section 3.5.1:

* the directory keeps, for the broadcast object, an ordered list of locations, each either
  complete or partial;
* a joining receiver is given ONE location: a complete copy if one can send, otherwise a
  partial one.  The chosen location stops being offered while it sends (here: it has ``d``
  send slots and one is taken; ``d = 1`` is the paper's rule) and the receiver is listed at
  once as a partial copy so that later receivers can fetch from it;
* when the receiver has the whole object it is marked complete and its sender gets the slot
  back;
* Section 3.5.1: when a sender fails its receivers query again and resume from the chunks
  they already hold; a candidate that (transitively) fetches from the receiver itself is
  not eligible, which keeps the dependencies acyclic.

Which transfers are still running when a receiver joins depends on time.  Time here is
virtual: one chunk crosses one edge in ``tau`` nanoseconds, a receiver fetches chunks in
order, one at a time, each as soon as its sender holds it:
``avail_r(c) = max(avail_sender(c), avail_r(c-1), t_join) + tau``.
Locations are offered oldest first (build-defined tie-break).
"""
from __future__ import annotations

import heapq
from dataclasses import dataclass, field

EDIT_REPARENT = 1   # orphan found a new sender
EDIT_WAIT = 2       # orphan found none and waits for a slot
EDIT_LEFT = 3       # a receiver left (its worker failed)


@dataclass
class Location:
    obj: int                  # object id of this copy (the source id for the original)
    order: int                # insertion order (0 = the source)
    have: int = 0             # chunks held
    complete: bool = False
    slots: int = 0            # free send slots
    alive: bool = True
    sender: "Location | None" = None
    first_sender_obj: int = -1
    start_chunk: int = 0      # first chunk fetched from the current sender
    t_join: int = -1
    t_complete: int = -1
    landing: int = -1         # virtual time at which the chunk in flight lands (-1: none)
    receivers: list = field(default_factory=list)


class BroadcastSchedule:
    def __init__(self, src_id: int, n_chunks: int, d: int, tau: int):
        self.src_id = src_id
        self.C = n_chunks
        self.d = d
        self.tau = tau
        self.now = 0
        self.source = Location(src_id, 0, slots=d, t_join=0)
        self.locs: list[Location] = [self.source]      # every location ever listed, in order
        self.by_obj: dict[int, Location] = {src_id: self.source}
        self.waiting: list[Location] = []              # receivers without a sender, first come first
        self.edits: list[list[int]] = []
        self.epoch = 0
        self._heap: list[tuple[int, int, int]] = []    # (landing time, order, token)
        self._token = 0
        self._tokens: dict[int, int] = {}              # order -> live token

    # ---- source progress (a Put that is still being copied is a partial location)
    def source_progress(self, t: int, have: int) -> None:
        self.advance(t)
        self.source.have = max(self.source.have, have)
        if self.source.have >= self.C and not self.source.complete:
            self.source.complete = True
            self.source.t_complete = t
        for r in list(self.source.receivers):
            self._try_start(r, t)

    # ---- virtual clock
    def advance(self, t: int) -> None:
        while self._heap and self._heap[0][0] <= t:
            tl, order, tok = heapq.heappop(self._heap)
            if self._tokens.get(order) != tok:
                continue   # cancelled transfer
            self._land(self.locs[order], tl)
        self.now = max(self.now, t)

    def _try_start(self, r: Location, t: int) -> None:
        if (not r.alive) or r.complete or r.landing >= 0 or r.sender is None:
            return
        if r.sender.have > r.have:
            r.landing = t + self.tau
            self._token += 1
            self._tokens[r.order] = self._token
            heapq.heappush(self._heap, (r.landing, r.order, self._token))

    def _land(self, r: Location, t: int) -> None:
        r.landing = -1
        r.have += 1
        if r.have >= self.C:
            r.complete = True
            r.t_complete = t
            s = r.sender
            if s is not None:
                s.receivers.remove(r)
                if s.alive:
                    s.slots += 1
            r.sender = None
            self._serve_waiting(t)
        else:
            self._try_start(r, t)
        for c in list(r.receivers):
            self._try_start(c, t)

    # ---- sender choice
    def _in_subtree(self, cand: Location, root: Location) -> bool:
        x = cand
        while x is not None:
            if x is root:
                return True
            x = x.sender
        return False

    def _choose(self, r: Location):
        best = None
        for loc in self.locs:
            if not loc.alive or loc is r or loc.slots <= 0:
                continue
            if self._in_subtree(loc, r):
                continue
            if loc.complete:
                return loc
            if best is None:
                best = loc
        return best

    def _attach(self, r: Location, s: Location, t: int) -> None:
        s.slots -= 1
        s.receivers.append(r)
        r.sender = s
        r.start_chunk = r.have
        self._try_start(r, t)

    def _serve_waiting(self, t: int) -> None:
        progressed = True
        while progressed:
            progressed = False
            for r in list(self.waiting):
                s = self._choose(r)
                if s is not None:
                    self.waiting.remove(r)
                    self._attach(r, s, t)
                    self.epoch += 1
                    self.edits.append([self.epoch, EDIT_REPARENT, r.obj, -1, s.obj, r.have, t])
                    progressed = True
                    break

    # ---- events
    def join(self, t: int, dst_obj: int) -> None:
        self.advance(t)
        if dst_obj in self.by_obj and self.by_obj[dst_obj].alive:
            return    # a request for this copy is already in flight: just wait for it
        # (a receiver whose worker failed and was rebuilt simply asks again, Section 3.5.1: a new location)
        r = Location(dst_obj, len(self.locs), slots=self.d, t_join=t)
        self.locs.append(r)
        self.by_obj[dst_obj] = r
        s = self._choose(r)
        if s is None:
            self.waiting.append(r)
        else:
            r.first_sender_obj = s.obj
            self._attach(r, s, t)
        self._serve_waiting(t)

    def fail(self, t: int, objs: list[int]) -> None:
        """The copies ``objs`` (all owned by one failed worker) disappear."""
        self.advance(t)
        gone = [self.by_obj[o] for o in objs if o in self.by_obj and self.by_obj[o].alive]
        gone.sort(key=lambda l: l.order)
        orphans: list[Location] = []
        for g in gone:
            g.alive = False
            self._tokens.pop(g.order, None)
            g.landing = -1
            if g in self.waiting:
                self.waiting.remove(g)
            s = g.sender
            if s is not None:
                if g in s.receivers:
                    s.receivers.remove(g)
                if s.alive:
                    s.slots += 1
                g.sender = None
            self.epoch += 1
            self.edits.append([self.epoch, EDIT_LEFT, g.obj, s.obj if s is not None else -1, -1, g.have, t])
            for c in g.receivers:
                orphans.append(c)
            g.receivers = []
        orphans = [o for o in orphans if o.alive]
        orphans.sort(key=lambda l: l.order)
        olds = []
        for o in orphans:          # every orphan first loses its sender and its chunk in flight ...
            self._tokens.pop(o.order, None)
            o.landing = -1
            olds.append(o.sender)
            o.sender = None
        for o, old in zip(orphans, olds):   # ... then each, oldest first, queries the directory again
            s = self._choose(o)
            self.epoch += 1
            if s is None:
                self.waiting.append(o)
                self.edits.append([self.epoch, EDIT_WAIT, o.obj, old.obj, -1, o.have, t])
            else:
                self._attach(o, s, t)
                self.edits.append([self.epoch, EDIT_REPARENT, o.obj, old.obj, s.obj, o.have, t])
        self._serve_waiting(t)

    # ---- serialisation (the word layout the library's schedule dump also produces)
    def words(self) -> list[int]:
        w = [0x48504C42, self.src_id, self.d, self.C, self.tau, self.now, len(self.locs) - 1]
        for r in self.locs[1:]:
            w += [r.obj, r.first_sender_obj, r.sender.obj if r.sender is not None else -1, r.start_chunk,
                  r.t_join, r.have, 1 if r.alive else 0, r.t_complete]
        w.append(len(self.edits))
        for e in self.edits:
            w += e
        return w
