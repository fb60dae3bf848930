"""Object store + directory driven by a timeline of events (Table 1 and Sections 3.1-3.5).

Test infrastructure (see the package docstring).  One instance stands for the whole cluster:
every object is one directory entry ``{size, owner, published prefix}`` (Section 3.2 keeps a
partial/complete bit per location; the prefix in chunks refines it, Section 3.3), a Reduce is a
:class:`ReduceSchedule` fed with arrivals and failures, a broadcast (many Gets of one id,
Section 3.4.1) is a :class:`BroadcastSchedule`.  Calls must come in timeline order (equal
times: failures, then publications, then requests).

"Arrival" of an object is its first publication, which Section 3.2 places at the moment Put is
called, before the copy has finished.

Composition (Sections 3.3, 3.4.2, 3.4.3): the output of a Reduce is an object like any other.  It is
published (as partial) when the Reduce is called, so it may be a source of a later Reduce or the
source of a broadcast (reduce followed by broadcast = allreduce); its chunk prefix is what its
current tree can already produce -- the smallest prefix among its members once the tree is full.
"""
from __future__ import annotations

import numpy as np

from .broadcast_tree import BroadcastSchedule
from .reduce_tree import ReduceSchedule, choose_degree
from .values import OP_SUM, tree_reduce

OK = 0
ERR_INVALID, ERR_NOT_FOUND, ERR_EXISTS, ERR_TIMEOUT, ERR_INSUFFICIENT, ERR_FAILED_WORKER = -1, -2, -3, -4, -5, -6

DT_F32, DT_BF16 = 0, 1
_ELEM = {DT_F32: 4, DT_BF16: 2}


class StoreError(Exception):
    def __init__(self, code: int, msg: str = ""):
        super().__init__(f"{code}: {msg}")
        self.code = code


class _Entry:
    def __init__(self, oid, worker, nbytes, dtype, chunk_bytes):
        self.oid, self.worker, self.nbytes, self.dtype = oid, worker, nbytes, dtype
        self.C = (nbytes + chunk_bytes - 1) // chunk_bytes
        self.elems = nbytes // _ELEM[dtype]
        self.chunk_elems = max(1, min(chunk_bytes, nbytes) // _ELEM[dtype])   # elements per chunk of this object
        self.data = None
        self.ready_bytes = 0
        self.alive = True
        self.arrived = False
        self.t_arrival = -1
        self.chunk_bytes = chunk_bytes

    @property
    def ready_chunks(self) -> int:
        return self.C if self.ready_bytes >= self.nbytes else self.ready_bytes // self.chunk_bytes

    @property
    def complete(self) -> bool:
        return self.ready_bytes >= self.nbytes


class OracleStore:
    def __init__(self, chunk_bytes: int, reduce_degree: int, bcast_degree: int, virt_chunk_ns: int = 0,
                 model_latency_ns: int = 0, model_bandwidth_bps: int = 0):
        self.chunk_bytes = chunk_bytes
        self.d_reduce = reduce_degree      # 0: chosen per Reduce by Eq. 1 from the two model parameters
        self.model_latency_ns = model_latency_ns
        self.model_bandwidth_bps = model_bandwidth_bps
        self.d_bcast = bcast_degree
        # default virtual chunk time: chunk_bytes at 64 GiB/s, in whole nanoseconds
        self.tau = virt_chunk_ns if virt_chunk_ns > 0 else max(1, chunk_bytes * 1_000_000_000 // (64 << 30))
        self.now = 0
        self.objects: dict[int, _Entry] = {}
        self.reduces: dict[int, dict] = {}       # target id -> {sched, op, srcs}
        self.bcasts: dict[int, dict] = {}        # source id -> {sched, dsts}
        self.dst_of: dict[int, int] = {}         # receiver id -> source id

    # ------------------------------------------------------------------ clock
    def advance(self, t_ns: int) -> None:
        if t_ns < self.now:
            raise StoreError(ERR_INVALID, "time goes forward")
        self.now = t_ns
        for b in self.bcasts.values():
            b["sched"].advance(t_ns)

    # ------------------------------------------------------------------ Table 1
    def create(self, oid: int, worker: int, nbytes: int, dtype: int) -> None:
        if oid in self.objects:
            raise StoreError(ERR_EXISTS)
        if nbytes <= 0 or nbytes % _ELEM[dtype]:
            raise StoreError(ERR_INVALID)
        self.objects[oid] = _Entry(oid, worker, nbytes, dtype, self.chunk_bytes)

    def put(self, oid: int, data: np.ndarray, nbytes: int) -> None:
        e = self._entry(oid)
        if not e.alive:
            raise StoreError(ERR_FAILED_WORKER)
        if oid in self.reduces or oid in self.dst_of:
            raise StoreError(ERR_INVALID, "produced by a collective")
        if nbytes < e.ready_bytes or nbytes > e.nbytes or data.nbytes != e.nbytes:
            raise StoreError(ERR_INVALID)
        first = not e.arrived
        e.data = data
        e.ready_bytes = nbytes
        if first:
            e.arrived = True
            e.t_arrival = self.now
            for r in self.reduces.values():
                if oid in r["srcs"]:
                    r["sched"].on_arrival(oid)
        if oid in self.bcasts:
            self.bcasts[oid]["sched"].source_progress(self.now, e.ready_chunks)
        self._refresh_composed()

    def reduce(self, target: int, srcs: list[int], k: int, op: int = OP_SUM, dtype: int = DT_F32) -> None:
        if target in self.objects:
            raise StoreError(ERR_EXISTS)
        n = len(srcs)
        if not (1 <= k <= n) or len(set(srcs)) != n:
            raise StoreError(ERR_INVALID)
        ents = [self._entry(s) for s in srcs]
        if any(e.dtype != dtype or e.nbytes != ents[0].nbytes or e.oid in self.dst_of for e in ents):
            raise StoreError(ERR_INVALID)
        live = [e for e in ents if e.alive]
        if len(live) < 1:
            raise StoreError(ERR_INSUFFICIENT)
        elems = ents[0].nbytes // _ELEM[dtype]
        self.create(target, -1, elems * 4, DT_F32)
        d = self.d_reduce
        if d == 0:
            d = choose_degree(k, float(ents[0].nbytes), self.model_latency_ns * 1e-9, float(self.model_bandwidth_bps))
        sched = ReduceSchedule(srcs, k, d)
        self.reduces[target] = {"sched": sched, "op": op, "srcs": list(srcs), "chunk_elems": ents[0].chunk_elems,
                                "C": ents[0].C}
        delivered = lambda o: self._delivered_in(o, target)
        for e in ents:                       # sources lost before the call never take part
            if not e.alive:
                sched.on_fail(e.oid, 0, delivered)
        arrived = sorted((e for e in live if e.arrived), key=lambda e: (e.t_arrival, srcs.index(e.oid)))
        for e in arrived:
            sched.on_arrival(e.oid)
        t = self.objects[target]          # the output is published at once, as a partial object
        t.arrived = True
        t.t_arrival = self.now
        self._refresh_composed()

    def broadcast(self, src: int, dsts: list[int]) -> None:
        e = self._entry(src)
        if src in self.bcasts:
            raise StoreError(ERR_EXISTS)
        for dd in dsts:
            de = self._entry(dd)
            if de.nbytes != e.nbytes or de.dtype != e.dtype or dd in self.dst_of or de.arrived or dd in self.reduces:
                raise StoreError(ERR_INVALID)
        sched = BroadcastSchedule(src, e.C, self.d_bcast, self.tau)
        sched.advance(self.now)
        if not e.alive:
            raise StoreError(ERR_FAILED_WORKER)
        if e.arrived:
            # chunks published before the broadcast existed count as available from now on
            sched.source_progress(self.now, self._delivered(src))
        self.bcasts[src] = {"sched": sched, "dsts": list(dsts)}
        for dd in dsts:
            self.dst_of[dd] = src

    def join(self, dst: int) -> None:
        if dst not in self.dst_of:
            raise StoreError(ERR_NOT_FOUND)
        if not self.objects[dst].alive:
            raise StoreError(ERR_FAILED_WORKER)
        self.bcasts[self.dst_of[dst]]["sched"].join(self.now, dst)

    def fail(self, worker: int) -> None:
        lost = [e for e in self.objects.values() if e.worker == worker and e.alive]
        for e in lost:
            e.alive = False
        for r in self.reduces.values():
            for e in lost:
                if e.oid in r["srcs"]:
                    tgt = next(t for t, rr in self.reduces.items() if rr is r)
                    r["sched"].on_fail(e.oid, self._delivered_in(e.oid, tgt), lambda o, tgt=tgt: self._delivered_in(o, tgt))
        for src, b in self.bcasts.items():
            mine = [e.oid for e in lost if e.oid == src or self.dst_of.get(e.oid) == src]
            if mine:
                b["sched"].fail(self.now, mine)
        self._refresh_composed()

    def rejoin(self, worker: int) -> None:
        """The task framework has reconstructed a failed worker (Section 3.5): its objects are futures again.
        A Reduce counts each as a new arrival once it is put again; a receiver may Get (join) again."""
        for e in self.objects.values():
            if e.worker == worker and not e.alive and e.oid not in self.bcasts:
                e.alive = True
                e.arrived = False
                e.data = None
                e.ready_bytes = 0
                e.t_arrival = -1
                for r in self.reduces.values():
                    if e.oid in r["srcs"]:
                        r["sched"].on_rejoin(e.oid)

    def delete(self, oid: int) -> None:
        self._entry(oid)
        if oid in self.dst_of or any(oid in r["srcs"] for r in self.reduces.values()):
            raise StoreError(ERR_INVALID, "still referenced")
        self.objects.pop(oid)
        if oid in self.reduces:
            self.reduces.pop(oid)
        if oid in self.bcasts:
            b = self.bcasts.pop(oid)
            for dd in b["dsts"]:      # Delete removes every copy of the object (Table 1): the receivers' copies go with it
                self.dst_of.pop(dd, None)
                self.objects.pop(dd, None)

    def get(self, oid: int) -> np.ndarray:
        """The complete object (read-only), or StoreError(ERR_TIMEOUT) if it cannot complete yet."""
        e = self._entry(oid)
        if oid in self.reduces:
            r = self.reduces[oid]
            sched: ReduceSchedule = r["sched"]
            if sched.k == 0:
                raise StoreError(ERR_INSUFFICIENT)
            if not sched.full() or any(self._ready_elems(m) < self.objects[m].elems for m in sched.members()):
                raise StoreError(ERR_TIMEOUT)
            key = self._membership(oid)
            if e.data is None or r.get("evaluated") != key:
                # a member that is itself the output of a Reduce is evaluated first (composed Reduce)
                objs = {m: (self.get(m) if m in self.reduces else self.objects[m].data) for m in sched.members()}
                e.data = tree_reduce(sched.obj_at, sched.d, objs, r["op"])
                r["evaluated"] = key
            return e.data
        if oid in self.dst_of:
            if not e.alive:
                raise StoreError(ERR_FAILED_WORKER)
            src = self.dst_of[oid]
            sched: BroadcastSchedule = self.bcasts[src]["sched"]
            loc = sched.by_obj.get(oid)
            if loc is None or not loc.alive:
                # never asked, or its worker was rebuilt and has not asked again (Section 3.5.1: a rebuilt receiver
                # fetches the object again as a new location; until then it holds no copy)
                raise StoreError(ERR_TIMEOUT, "has not joined")
            # blocking on the copy = letting virtual time run until it has landed
            while not loc.complete and sched._heap:
                sched.advance(sched._heap[0][0])
            if not loc.complete:
                raise StoreError(ERR_TIMEOUT)
            self.now = max(self.now, sched.now)
            for b in self.bcasts.values():
                b["sched"].advance(self.now)
            srcdata = self.get(src) if src in self.reduces else self.objects[src].data
            if e.data is None or src in self.reduces:
                e.data = srcdata.copy()
                e.ready_bytes = e.nbytes
            return e.data
        if not e.alive:
            raise StoreError(ERR_FAILED_WORKER)
        if not e.complete:
            raise StoreError(ERR_TIMEOUT)
        return e.data

    # ------------------------------------------------------------------ schedule dump
    def dump(self, op_id: int) -> list[int]:
        if op_id in self.reduces:
            return self.reduces[op_id]["sched"].words(op_id)
        if op_id in self.bcasts:
            return self.bcasts[op_id]["sched"].words()
        if op_id in self.dst_of:          # a receiver names the broadcast it belongs to
            return self.bcasts[self.dst_of[op_id]]["sched"].words()
        raise StoreError(ERR_NOT_FOUND)

    # ------------------------------------------------------------------ helpers
    def _entry(self, oid: int) -> _Entry:
        if oid not in self.objects:
            raise StoreError(ERR_NOT_FOUND)
        return self.objects[oid]

    def _ready_elems(self, oid: int) -> int:
        """Published element prefix: of a Put object what was put (whole chunks); of a Reduce output what its
        tree can produce, i.e. the smallest prefix among its members once the tree is full."""
        e = self.objects[oid]
        if oid in self.reduces:
            sched = self.reduces[oid]["sched"]
            if not sched.full():
                return 0
            return min(self._ready_elems(m) for m in sched.members())
        return e.elems if e.complete else e.ready_chunks * e.chunk_elems

    def _delivered(self, oid: int) -> int:
        """The same prefix counted in the object's own chunks (chunk_bytes of its own dtype)."""
        e = self.objects[oid]
        n = self._ready_elems(oid)
        return e.C if n >= e.elems else n // e.chunk_elems

    def _delivered_in(self, oid: int, target: int) -> int:
        """The same prefix counted in the chunks of the Reduce that produces ``target`` (chunk_bytes of its
        input dtype: a bf16 Reduce works on twice as many elements per chunk as its fp32 output holds)."""
        r = self.reduces[target]
        n = self._ready_elems(oid)
        return r["C"] if n >= self.objects[oid].elems else n // r["chunk_elems"]

    def _membership(self, oid: int) -> tuple:
        """Who is in the tree of ``oid``, and in the trees of the members that are Reduce outputs themselves."""
        sched = self.reduces[oid]["sched"]
        return tuple(sched.obj_at) + tuple(self._membership(m) for m in sched.members() if m in self.reduces)

    def _refresh_composed(self) -> None:
        """After every event: a broadcast whose source is a Reduce output learns how far that output has got."""
        for src, b in self.bcasts.items():
            if src in self.reduces:
                b["sched"].source_progress(self.now, self._delivered(src))
