"""Every call's refusals, on a schedule-only context (no GPU): the code the header gives, and nothing changed by the
refused call (the schedule dump before and after is the same)."""
import ctypes

import pytest

import paper_2002_05814_b200 as hpl
from paper_2002_05814_b200 import build as hpl_build

S = 4096


@pytest.fixture(scope="module", autouse=True)
def _built():
    hpl_build.build()


def _code(call, *a, **kw):
    with pytest.raises(hpl.HplError) as e:
        call(*a, **kw)
    return e.value.code


def _ctx():
    c = hpl.Context(1024, 2, 2)
    for i in range(6):
        c.create(i, i, S)
    c.create(20, 6, S, hpl.HPL_BF16)
    c.create(21, 6, 2 * S)
    for j in range(3):
        c.create(50 + j, 10 + j, S)
    return c


def test_reduce_refusals():
    c = _ctx()
    I = hpl.HPL_ERR_INVALID
    assert _code(c.reduce, 100, [0, 1], 3) == I                         # k > n
    assert _code(c.reduce, 100, [0, 1], 0) == I
    assert _code(c.reduce, 100, [], 1) == I
    assert _code(c.reduce, 100, [0, 0], 1) == I                         # the same object twice
    assert _code(c.reduce, 100, [0, 20], 2) == I                        # dtypes differ
    assert _code(c.reduce, 100, [0, 21], 2) == I                        # sizes differ
    assert _code(c.reduce, 100, [0, 1], 2, 7) == I                      # no such operator
    assert _code(c.reduce, 100, [0, 1], 2, hpl.HPL_SUM, 5) == I         # no such dtype
    assert _code(c.reduce, 100, [0, 99], 2) == hpl.HPL_ERR_NOT_FOUND
    assert _code(c.reduce, 0, [1, 2], 2) == hpl.HPL_ERR_EXISTS
    assert _code(c.reduce, -3, [1, 2], 2) == I
    c.broadcast(0, [50, 51])
    assert _code(c.reduce, 100, [1, 50], 2) == I                        # a receiver copy is no source
    c.fail(1)
    c.fail(2)
    assert _code(c.reduce, 100, [1, 2], 2) == hpl.HPL_ERR_INSUFFICIENT  # no live source
    c.reduce(100, [1, 2, 3], 3)                                         # lost sources never take part: the tree has one position
    assert c.schedule_dump(100)[4] == 1
    assert _code(c.reduce, 100, [3, 4], 2) == hpl.HPL_ERR_EXISTS
    assert c.stats()["arena_used"] == S                                 # the one output; no refused call left anything behind
    c.shutdown()


def test_broadcast_and_join_refusals():
    c = _ctx()
    I = hpl.HPL_ERR_INVALID
    assert _code(c.broadcast, 99, [50]) == hpl.HPL_ERR_NOT_FOUND
    assert _code(c.broadcast, 0, [98]) == hpl.HPL_ERR_NOT_FOUND
    assert _code(c.broadcast, 0, []) == I
    assert _code(c.broadcast, 0, [50, 50]) == I
    assert _code(c.broadcast, 0, [21]) == I                             # another size
    assert _code(c.broadcast, 0, [20]) == I                             # another dtype
    c.put(1, 1 << 20, S)
    assert _code(c.broadcast, 0, [1]) == I                              # has a value of its own already
    assert _code(c.join, 50, 1 << 21) == hpl.HPL_ERR_NOT_FOUND          # no receiver of that name (yet)
    c.broadcast(0, [50, 51])
    before = c.schedule_dump(0)
    assert _code(c.broadcast, 0, [52]) == hpl.HPL_ERR_EXISTS            # one broadcast per source
    assert _code(c.broadcast, 2, [50]) == I                             # already a receiver of another broadcast
    assert _code(c.join, 97, 1 << 21) == hpl.HPL_ERR_NOT_FOUND
    assert _code(c.join, 0, 1 << 21) == hpl.HPL_ERR_NOT_FOUND
    assert _code(c.put, 50, 1 << 22, S) == I                            # a receiver is filled by the broadcast only
    assert _code(c.delete, 50) == I                                     # goes with its broadcast
    assert c.schedule_dump(0) == before
    c.fail(0)                                                           # the source is lost
    assert _code(c.broadcast, 0, [52]) in (hpl.HPL_ERR_EXISTS, hpl.HPL_ERR_FAILED_WORKER)
    c.fail(2)
    assert _code(c.broadcast, 2, [52]) == hpl.HPL_ERR_FAILED_WORKER
    c.shutdown()


def test_put_get_delete_and_clock_refusals():
    c = _ctx()
    I = hpl.HPL_ERR_INVALID
    assert _code(c.create, 0, 0, S) == hpl.HPL_ERR_EXISTS
    assert _code(c.create, 70, -1, S) == I
    assert _code(c.create, 70, 0, 0) == I
    assert _code(c.create, 70, 0, S + 2) == I                           # not a whole number of fp32 elements
    assert _code(c.create, 70, 0, S, 9) == I
    assert _code(c.create, -1, 0, S) == I
    assert _code(c.put, 0, 0, S) == I                                   # null buffer
    assert _code(c.put, 0, 1 << 20, S + 16) == I                        # longer than the object
    c.put(0, 1 << 20, 2048)
    assert _code(c.put, 0, 1 << 21, S) == I                             # another buffer for the same object
    assert _code(c.put, 0, 1 << 20, 1024) == I                          # the prefix never shrinks
    c.put(0, 1 << 20, 2048)                                             # the same prefix again is no event
    c.fail(1)
    assert _code(c.put, 1, 1 << 20, S) == hpl.HPL_ERR_FAILED_WORKER
    assert c.try_get(98)[0] == hpl.HPL_ERR_NOT_FOUND
    assert c.try_get(0)[0] == hpl.HPL_ERR_TIMEOUT                       # partial
    assert c.try_get(2)[0] == hpl.HPL_ERR_TIMEOUT                       # a future
    assert c.try_get(1)[0] == hpl.HPL_ERR_FAILED_WORKER
    c.reduce(100, [0, 2], 2)
    assert _code(c.delete, 0) == I                                      # still a source of a Reduce
    assert _code(c.delete, 98) == hpl.HPL_ERR_NOT_FOUND
    c.delete(100)
    c.delete(0)
    assert c.try_get(0)[0] == hpl.HPL_ERR_NOT_FOUND
    c.advance(100)
    assert _code(c.advance, 99) == I
    c.advance(100)
    assert _code(c.fail, -1) == I
    assert _code(c.rejoin, -1) == I
    c.fail(77)                                                          # a worker that owns nothing: no event
    c.rejoin(77)
    c.shutdown()


def test_calls_of_the_other_modes_and_helpers():
    c = _ctx()
    I = hpl.HPL_ERR_INVALID
    assert _code(c.set_peer_arena, 1, 1 << 30) == I            # one GPU: there are no peers
    assert _code(c.fail_rank, 1) == I
    assert c.pending_levels() == 0
    assert _code(hpl.Context, 1024, 2, 2, rank=2, world_size=2) == I
    assert _code(hpl.Context, 1024, 2, 2, rank=0, world_size=2, eager=True) == I
    assert _code(hpl.Context, 1024, 2, 2, rank=0, world_size=2, plan_ahead=True) == I
    assert _code(hpl.Context, 1024, 0, 2) == I                          # degree chosen by the model needs the model
    assert _code(hpl.Context, 1024, 2, 0) == I
    assert _code(hpl.Context, 0, 2, 2) == I
    lib = hpl.load_library()
    assert lib.hpl_choose_degree(0, 1024, ctypes.c_double(1e-6), ctypes.c_double(1e9)) == I
    assert lib.hpl_choose_degree(8, 1024, ctypes.c_double(1e-6), ctypes.c_double(0.0)) == I
    assert lib.hpl_choose_degree(1, 1024, ctypes.c_double(1e-6), ctypes.c_double(1e9)) == 1
    n = ctypes.c_size_t(0)
    assert lib.hpl_schedule_dump(c._h, 12345, None, 0, ctypes.byref(n)) == hpl.HPL_ERR_NOT_FOUND
    c.reduce(100, [0, 1], 2)
    assert lib.hpl_schedule_dump(c._h, 100, None, 0, ctypes.byref(n)) == I and n.value > 0   # too small: says how many
    buf = (ctypes.c_int64 * n.value)()
    assert lib.hpl_schedule_dump(c._h, 100, buf, n.value, ctypes.byref(n)) == 0
    for f in (lib.hpl_progress, lib.hpl_sync, lib.hpl_shutdown):
        assert f(None) == I
    c.shutdown()


def test_an_object_named_by_several_reduces_is_held_until_the_last_one_is_deleted():
    c = _ctx()
    I = hpl.HPL_ERR_INVALID
    c.reduce(100, [0, 1], 2)
    c.reduce(101, [1, 2], 2)
    c.reduce(102, [1, 3, 4], 2)
    c.put(1, 1 << 20, S)                                # one arrival, noted by all three trees, in the order of their requests
    for tgt in (100, 101, 102):
        assert 1 in c.schedule_dump(tgt)[7:9]           # the first placement: (object 1, its position)
    assert _code(c.delete, 1) == I
    c.delete(101)
    assert _code(c.delete, 1) == I
    c.delete(100)
    assert _code(c.delete, 1) == I                      # 102 still names it
    c.put(3, 1 << 21, S)
    c.delete(102)
    c.delete(1)
    c.delete(3)
    assert c.try_get(1)[0] == hpl.HPL_ERR_NOT_FOUND
    c.shutdown()
