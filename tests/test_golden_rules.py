"""Hand-worked timelines (tests/golden/) for the rules the paper leaves open and this build fixes: how a
prefix crosses dtypes in composed collectives, what a reduce tree looks like after it shrinks, which
sender a receiver is given when several locations can send, and in which order waiting receivers are
served.  The expected numbers were worked out by hand from the wording of the rules; the oracle AND
the library's schedule builders (a schedule-only context, no GPU) are each held to them, so that
their agreement with one another is not the only evidence."""
import numpy as np
import pytest

import paper_2002_05814_b200 as hpl
from oracle.store import OracleStore, DT_F32, DT_BF16
from paper_2002_05814_b200 import build as hpl_build
from tests.conftest import read_golden


@pytest.fixture(scope="module", autouse=True)
def _built():
    hpl_build.build()


# ------------------------------------------------------------------ reading a schedule dump (layout: include/hpl.h)
def parse_reduce(w):
    assert w[0] == 0x48504C52
    out = {"target": w[1], "n": w[2], "k0": w[3], "k": w[4], "d": w[5]}
    i = 7
    out["placements"] = [(w[i + 2 * j], w[i + 2 * j + 1]) for j in range(w[6])]
    i += 2 * w[6]
    out["obj_at"] = list(w[i:i + out["k"]])
    i += out["k"]
    out["parent"] = list(w[i:i + out["k"]])
    i += out["k"]
    ns = w[i]
    out["spares"] = list(w[i + 1:i + 1 + ns])
    i += 1 + ns
    edits = []
    for _ in range(w[i]):
        e = dict(zip(("epoch", "kind", "pos", "old", "new", "moved_from", "hi_failed", "hi_moved"), w[i + 1:i + 9]))
        nc = w[i + 9]
        e["cleared"] = list(w[i + 10:i + 10 + nc])
        edits.append(e)
        i += 9 + nc
    out["edits"] = edits
    return out


def parse_bcast(w):
    assert w[0] == 0x48504C42
    out = {"src": w[1], "d": w[2], "C": w[3], "tau": w[4], "now": w[5], "recv": {}, "order": []}
    i = 7
    for _ in range(w[6]):
        r = dict(zip(("id", "first_sender", "sender", "start_chunk", "t_join", "have", "alive", "t_complete"), w[i:i + 8]))
        out["recv"][r["id"]] = r
        out["order"].append(r["id"])
        i += 8
    out["edits"] = [dict(zip(("epoch", "kind", "recv", "old", "new", "have", "t"), w[i + 1 + 7 * j:i + 8 + 7 * j])) for j in range(w[i])]
    return out


def edit_words(e):
    return (f"epoch {e['epoch']} kind {e['kind']} pos {e['pos']} old {e['old']} new {e['new']} moved_from {e['moved_from']} "
            f"hi_failed {e['hi_failed']} hi_moved {e['hi_moved']} cleared " + " ".join(str(c) for c in e["cleared"])).strip()


def ints(s):
    return [int(x) for x in s.split()]


class Both:
    """The same events to the oracle's store and to a schedule-only library context."""

    def __init__(self, chunk, d_reduce, d_bcast, tau):
        self.o = OracleStore(chunk, d_reduce, d_bcast, tau)
        self.c = hpl.Context(chunk, d_reduce, d_bcast, virt_chunk_ns=tau)
        self.data = {}

    def close(self):
        self.c.shutdown()

    def advance(self, t):
        self.o.advance(t)
        self.c.advance(t)

    def create(self, oid, worker, data=None, nbytes=None, dtype=DT_F32):
        if data is not None:
            self.data[oid] = data
            nbytes = data.nbytes
            dtype = DT_BF16 if data.dtype == np.uint16 else DT_F32
        self.o.create(oid, worker, nbytes, dtype)
        self.c.create(oid, worker, nbytes, dtype)

    def put(self, oid, nbytes=None):
        nbytes = self.data[oid].nbytes if nbytes is None else nbytes
        self.o.put(oid, self.data[oid], nbytes)
        self.c.put(oid, 4096 * (oid + 1), nbytes)      # a schedule-only context never dereferences the address

    def reduce(self, target, srcs, k, dtype=DT_F32):
        self.o.reduce(target, srcs, k, 0, dtype)
        self.c.reduce(target, srcs, k, 0, dtype)

    def broadcast(self, src, dsts):
        self.o.broadcast(src, dsts)
        self.c.broadcast(src, dsts)

    def join(self, dst):
        self.o.join(dst)
        self.c.join(dst, None)

    def fail(self, worker):
        self.o.fail(worker)
        self.c.fail(worker)

    def dumps(self, op_id, parse):
        """The schedule of ``op_id`` as each side serialises it, parsed."""
        return parse(self.o.dump(op_id)), parse(self.c.schedule_dump(op_id))


def bf16_bits(a):
    """Small integers as bf16 bit patterns (exact: they need at most 8 significant bits)."""
    return (np.asarray(a, np.float32).view(np.uint32) >> 16).astype(np.uint16)


# ------------------------------------------------------------------ composition across dtypes (Sections 3.3, 3.4.2, 3.4.3)
def test_prefixes_cross_dtypes_in_elements_and_are_counted_in_each_consumers_chunks():
    g = read_golden("composition_cross_dtype.txt")
    rng = np.random.default_rng(5)
    b = Both(64, 2, 1, 1)
    for oid in (0, 1, 2, 5):
        b.create(oid, 10 + oid, bf16_bits(rng.integers(0, 8, 80)))
    for oid in (3, 4):
        b.create(oid, 10 + oid, rng.integers(0, 8, 80).astype(np.float32))
    for r in (300, 301):
        b.create(r, r, nbytes=320, dtype=DT_F32)
    A, B = 100, 200
    b.advance(1)
    b.put(3)
    b.put(4, 192)
    b.advance(2)
    b.reduce(A, [0, 1, 2, 5], 3, DT_BF16)
    b.reduce(B, [3, 4, A], 3, DT_F32)
    b.broadcast(B, [300, 301])
    b.join(300)
    for side in b.dumps(B, parse_reduce):
        assert side["obj_at"] == ints(g["b_positions_at_t2"])
    b.advance(3)
    b.put(0)
    b.put(1)
    b.put(2, 128)
    o = b.o
    assert o._ready_elems(A) == int(g["ready_elems_100_at_t3"])
    assert o._delivered(A) == int(g["delivered_100_at_t3"])
    assert o._delivered_in(2, A) == int(g["delivered_2_in_A_at_t3"])
    assert o._delivered_in(A, B) == int(g["delivered_100_in_B_at_t3"])
    assert o._ready_elems(B) == int(g["ready_elems_200_at_t3"])
    assert o._delivered(B) == int(g["delivered_200_at_t3"])
    b.advance(4)
    b.put(4)
    assert o._delivered(B) == int(g["delivered_200_at_t4"])
    b.advance(20)
    for side in b.dumps(300, parse_bcast):    # what the broadcast of the second output has seen of its source
        assert side["recv"][300]["have"] == int(g["receiver_300_chunks_at_t20"])
    b.advance(21)
    b.fail(12)
    for side in b.dumps(A, parse_reduce):
        assert [edit_words(e) for e in side["edits"]] == [g["a_edit_1"]]
    assert o._ready_elems(A) == int(g["ready_elems_100_at_t21"]) and o._ready_elems(B) == int(g["ready_elems_200_at_t21"])
    b.advance(22)
    b.put(5, 64)
    assert o._delivered(A) == int(g["delivered_100_at_t22"]) and o._delivered(B) == int(g["delivered_200_at_t22"])
    b.advance(23)
    b.fail(13)
    for side in b.dumps(B, parse_reduce):
        assert [edit_words(e) for e in side["edits"]] == [g["b_edit_1"]]
        assert side["obj_at"] == ints(g["b_positions_at_t23"])
    b.advance(24)
    b.put(5)
    b.join(301)
    from oracle.values import widen
    want_a = sum(widen(b.data[i]) for i in ints(g["final_100"]))
    want_b = sum(widen(b.data[i]) for i in ints(g["final_200"]))
    assert np.array_equal(o.get(A), want_a) and np.array_equal(o.get(B), want_b)
    for r in (300, 301):
        assert o.get(r).tobytes() == want_b.astype(np.float32).tobytes()
    b.close()


def test_a_planted_chunk_mistake_in_the_oracle_fails_the_composition_pin(monkeypatch):
    """The pin has teeth: counting a Reduce output's prefix in the producing Reduce's chunks instead of the
    consumer's (the plausible slip) changes the numbers the golden file fixes."""
    g = read_golden("composition_cross_dtype.txt")
    o = OracleStore(64, 2, 1, 1)
    for oid in (0, 1, 2):
        o.create(oid, oid, 160, DT_BF16)
    o.reduce(100, [0, 1, 2], 3, 0, DT_BF16)
    z = np.zeros(80, np.uint16)
    o.put(0, z, 160)
    o.put(1, z, 160)
    o.put(2, z, 128)
    assert o._delivered(100) == int(g["delivered_100_at_t3"])
    wrong = lambda oid: o._ready_elems(oid) // o.reduces[100]["chunk_elems"]     # the producer's bf16 chunks
    assert wrong(100) != int(g["delivered_100_at_t3"])


# ------------------------------------------------------------------ reduce tree after a shrink (build-defined)
def test_shrink_moves_the_last_position_into_the_opening():
    g = read_golden("reduce_shrink_example.txt")
    rng = np.random.default_rng(6)
    b = Both(64, 2, 1, 1)
    for oid in range(6):
        b.create(oid, 20 + oid, rng.integers(-8, 8, 64).astype(np.float32))     # 256 bytes = 4 chunks
    b.reduce(100, list(range(6)), 6)
    for oid in range(6):
        b.advance(oid + 1)
        b.put(oid, {1: 128, 4: 192}.get(oid))
    for side in b.dumps(100, parse_reduce):
        assert side["obj_at"] == ints(g["positions_initial"])
    for n, worker in enumerate((21, 22, 23), start=1):
        b.advance(10 + n)
        b.fail(worker)
        for side in b.dumps(100, parse_reduce):
            assert edit_words(side["edits"][-1]) == g[f"edit_{n}"] and len(side["edits"]) == n
            assert side["obj_at"] == ints(g[f"positions_after_{n}"])
            assert side["parent"] == [-1 if p == 0 else (p - 1) // 2 for p in range(len(side["obj_at"]))]
    b.advance(20)
    b.put(4)
    assert np.array_equal(b.o.get(100), sum(b.data[i] for i in ints(g["final_members"])))
    b.close()


# ------------------------------------------------------------------ broadcast with two send slots (build-defined)
def test_oldest_complete_copy_with_a_free_slot_else_oldest_partial():
    g = read_golden("broadcast_two_slots_example.txt")
    name = lambda oid: "S" if oid == 0 else f"R{oid}"
    b = Both(64, 2, 2, 10)
    b.create(0, 99, np.arange(64, dtype=np.float32))
    for r in range(1, 13):
        b.create(r, r, nbytes=256)
    b.put(0)
    b.broadcast(0, list(range(1, 13)))
    for t, rs in ((0, (1, 2, 3)), (5, (4, 5, 6, 7)), (45, (8, 9, 10, 11)), (55, (12,))):
        b.advance(t)
        for r in rs:
            b.join(r)
    b.advance(100)
    for side in b.dumps(0, parse_bcast):
        assert " ".join(f"{name(r)}:{name(side['recv'][r]['first_sender'])}" for r in side["order"]) == g["first_sender"]
        assert " ".join(f"{name(r)}:{side['recv'][r]['t_complete']}" for r in side["order"]) == g["completed_at"]
        assert side["edits"] == []
    b.close()


# ------------------------------------------------------------------ orphans of one failure (build-defined)
def test_orphans_all_lose_their_sender_before_any_asks_again_and_one_may_have_to_wait():
    g = read_golden("broadcast_orphans_example.txt")
    b = Both(64, 2, 1, 10)
    b.create(0, 60, np.arange(128, dtype=np.float32))      # 512 bytes = 8 chunks
    for r, wk in ((1, 60), (2, 70), (3, 60), (4, 71)):
        b.create(r, wk, nbytes=512)
    b.put(0)
    b.broadcast(0, [1, 2, 3, 4])
    for t, r in enumerate((1, 2, 3, 4)):
        b.advance(t)
        b.join(r)
    b.advance(45)
    b.fail(60)
    want = [ints(rec) for rec in g["edits"].split("|")]
    b.advance(500)
    for side in b.dumps(2, parse_bcast):
        assert [[e[k] for k in ("epoch", "kind", "recv", "old", "new", "have", "t")] for e in side["edits"]] == want
        assert " ".join(f"{r}:{side['recv'][r]['sender']}" for r in (2, 4)) == g["sender_after"]
        assert " ".join(f"{r}:{side['recv'][r]['have']}" for r in (2, 4)) == g["have_after"]
    b.close()
