"""hpl_submit on a schedule-only context (no GPU): a timeline handed over in one call is applied exactly like the single
calls -- same schedules, same codes -- stops at the first event that fails and says how many were applied."""
import numpy as np
import pytest

import paper_2002_05814_b200 as hpl
from paper_2002_05814_b200 import build as hpl_build


@pytest.fixture(scope="module", autouse=True)
def _built():
    hpl_build.build()


S = 5 * 4096 + 64


def _single_calls(c):
    for i in range(6):
        c.create(i, i, S)
    for j in range(3):
        c.create(50 + j, 20 + j, S)
    c.reduce(100, list(range(6)), 4)
    c.broadcast(100, [50, 51, 52])
    for t, i in enumerate([3, 0, 5, 1, 4]):
        c.advance(10 * (t + 1))
        c.put(i, 4096 * (i + 1), S if i != 5 else 4096)
    c.advance(100)
    c.join(50, None)
    c.fail(0)
    c.advance(200)
    c.join(51, None)
    c.progress()


def _timeline():
    H = hpl
    e = hpl.EventList(64)
    for i in range(6):
        e.add(H.HPL_EV_CREATE, 0, i, i, nbytes=S)
    for j in range(3):
        e.add(H.HPL_EV_CREATE, 0, 50 + j, 20 + j, nbytes=S)
    e.add(H.HPL_EV_REDUCE, 0, 100, ids=list(range(6)), k=4)
    e.add(H.HPL_EV_BROADCAST, 0, 100, ids=[50, 51, 52])
    for t, i in enumerate([3, 0, 5, 1, 4]):
        e.add(H.HPL_EV_PUT, 10 * (t + 1), i, ptr=4096 * (i + 1), nbytes=S if i != 5 else 4096)
    e.add(H.HPL_EV_JOIN, 100, 50)
    e.add(H.HPL_EV_FAIL, 0, worker=0)                    # t_ns = 0: the clock stays where it is
    e.add(H.HPL_EV_JOIN, 200, 51)
    e.add(H.HPL_EV_PROGRESS)
    return e


def test_a_timeline_in_one_call_equals_the_single_calls():
    with hpl.Context(4096, 2, 2) as a, hpl.Context(4096, 2, 2) as b:
        _single_calls(a)
        b.submit(_timeline())
        assert a.schedule_dump(100) == b.schedule_dump(100)
        assert a.schedule_dump(50) == b.schedule_dump(50)          # a receiver names its broadcast
        sa, sb = a.stats(), b.stats()
        for key in ("reduce_tasks", "fanout_tasks", "bytes_read_planned", "bytes_written_planned", "kernel_launches"):
            assert sa[key] == sb[key], key


def test_submit_stops_at_the_first_failing_event_and_counts_the_applied_ones():
    H = hpl
    with hpl.Context(4096, 2, 2) as c:
        e = hpl.EventList(8)
        e.add(H.HPL_EV_CREATE, 5, 1, 1, nbytes=64)
        e.add(H.HPL_EV_CREATE, 5, 1, 1, nbytes=64)       # the id exists already
        e.add(H.HPL_EV_CREATE, 5, 2, 2, nbytes=64)
        with pytest.raises(hpl.HplError) as ei:
            c.submit(e)
        assert ei.value.code == hpl.HPL_ERR_EXISTS and "event 1 of 3" in str(ei.value)
        assert c.try_get(2)[0] == hpl.HPL_ERR_NOT_FOUND                 # the third event was not applied
        back = hpl.EventList(2)
        back.add(H.HPL_EV_CREATE, 3, 9, 9, nbytes=64)    # time going back
        with pytest.raises(hpl.HplError) as ei:
            c.submit(back)
        assert ei.value.code == hpl.HPL_ERR_INVALID and "event 0 of 1" in str(ei.value)
        bad = hpl.EventList(2)
        bad.add(99)                                      # no such kind
        with pytest.raises(hpl.HplError) as ei:
            c.submit(bad)
        assert ei.value.code == hpl.HPL_ERR_INVALID
        g = hpl.EventList(2)
        g.add(H.HPL_EV_PUT, 0, 1, ptr=4096, nbytes=64)
        g.add(H.HPL_EV_GET, 0, 1)
        with pytest.raises(hpl.HplError) as ei:          # complete, but a schedule-only context has no device to wait for
            c.submit(g)
        assert ei.value.code == hpl.HPL_ERR_CUDA and "event 1 of 2" in str(ei.value)
        assert c.submit(hpl.EventList(1)) is None        # an empty timeline is fine
