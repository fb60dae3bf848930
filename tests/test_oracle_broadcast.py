"""Pins for the broadcast half of the oracle: the paper's worked example with and without a
failure, virtual-time closed forms, and invariants under random joins and failures."""
import numpy as np
import pytest

from oracle.broadcast_tree import BroadcastSchedule, EDIT_REPARENT
from oracle.store import OracleStore, StoreError, ERR_TIMEOUT, DT_F32
from tests.conftest import read_golden

S, R1, R2, R3 = 0, 1, 2, 3
NAMES = {S: "S", R1: "R1", R2: "R2", R3: "R3"}


def _pairs(text):
    return dict(p.split(":") for p in text.split())


def _example(tau=10, C=8):
    b = BroadcastSchedule(S, C, 1, tau)
    b.source_progress(0, C)            # the Put has completed before anyone asks
    return b


def test_paper_example_fig4_without_failure():
    g = _pairs(read_golden("broadcast_example.txt")["senders"])
    b = _example()
    b.join(0, R1)                                   # (a)
    b.join(25, R2)                                  # (b) S still sends to R1 (until t = 80)
    assert b.by_obj[R2].sender is b.by_obj[R1]
    b.advance(85)                                   # (c) R1 complete, still sending to R2
    listed = [(NAMES[l.obj], l.complete) for l in b.locs if l.alive and l.slots > 0]
    assert listed == [("S", True), ("R2", False)]
    b.join(85, R3)                                  # (d) complete beats partial
    got = {NAMES[r.obj]: NAMES[r.first_sender_obj] for r in b.locs[1:]}
    assert got == g


def test_paper_example_fig4_with_r1_failing():
    g = _pairs(read_golden("broadcast_example.txt")["senders_after_R1_fails"])
    b = _example()
    b.join(0, R1)
    b.join(25, R2)
    b.advance(52)
    have = b.by_obj[R2].have
    assert 0 < have < b.C
    b.fail(52, [R1])                                # (c') R2 asks again and resumes from S
    r2 = b.by_obj[R2]
    assert NAMES[r2.sender.obj] == g["R2"] and r2.start_chunk == have   # only the rest is sent
    b.join(60, R3)                                  # (d') S is busy with R2: R3 fetches from R2
    assert NAMES[b.by_obj[R3].sender.obj] == g["R3"]
    b.advance(10_000)
    assert b.by_obj[R2].complete and b.by_obj[R3].complete
    assert [e[1] for e in b.edits].count(EDIT_REPARENT) == 1


# ---------------------------------------------------------------- virtual-time closed forms
def test_chain_completion_times_when_all_join_at_once():
    C, tau, R = 16, 7, 6
    b = BroadcastSchedule(0, C, 1, tau)
    b.source_progress(0, C)
    for j in range(1, R + 1):
        b.join(0, j)
    b.advance(10**9)
    for j in range(1, R + 1):        # chunk c reaches the j-th receiver of a chain at (c + j) * tau
        assert b.by_obj[j].t_complete == (C - 1 + j) * tau
        assert b.by_obj[j].first_sender_obj == j - 1


def test_slow_joins_all_fetch_from_the_source():
    C, tau = 4, 5
    b = BroadcastSchedule(0, C, 1, tau)
    b.source_progress(0, C)
    for j in range(1, 6):
        b.join(j * 100, j)           # each join comes after the previous transfer has finished
        assert b.by_obj[j].first_sender_obj == 0
    b.advance(10**6)
    assert [b.by_obj[j].t_complete for j in range(1, 6)] == [j * 100 + C * tau for j in range(1, 6)]


@pytest.mark.parametrize("d", [1, 2, 3, 4])
def test_all_at_once_gives_the_heap_ordered_tree(d):
    b = BroadcastSchedule(0, 8, d, 3)
    b.source_progress(0, 8)
    for j in range(1, 30):
        b.join(0, j)
    for j in range(1, 30):
        assert b.by_obj[j].first_sender_obj == (j - 1) // d


def test_partial_source_paces_everyone():
    C, tau = 6, 4
    b = BroadcastSchedule(0, C, 2, tau)
    b.source_progress(0, 1)
    b.join(0, 1)
    b.join(0, 2)
    b.advance(50)
    assert b.by_obj[1].have == 1 and not b.by_obj[1].complete
    b.source_progress(100, C)
    b.advance(10**6)
    assert b.by_obj[1].t_complete == 100 + (C - 1) * tau


# ---------------------------------------------------------------- invariants under random timelines
def _check_invariants(b: BroadcastSchedule):
    for loc in b.locs:
        if not loc.alive:
            continue
        sending = [r for r in loc.receivers if r.alive and not r.complete]
        assert len(sending) + loc.slots == b.d            # one slot per running send (Section 3.4.1)
        seen, x = set(), loc
        while x is not None:                              # the sender chain ends: no cycle (Section 3.5.1)
            assert id(x) not in seen
            seen.add(id(x))
            x = x.sender
        if loc.sender is not None:
            assert loc.sender.alive and loc.have <= max(loc.sender.have, loc.have)
        assert 0 <= loc.have <= b.C and loc.complete == (loc.have >= b.C or (loc is b.source and loc.complete))


def test_random_joins_and_failures_keep_invariants_and_finish():
    rng = np.random.default_rng(31)
    for trial in range(200):
        C = int(rng.integers(1, 12))
        d = int(rng.integers(1, 4))
        tau = int(rng.integers(1, 20))
        R = int(rng.integers(1, 14))
        b = BroadcastSchedule(0, C, d, tau)
        b.source_progress(0, C)
        events = sorted([(int(rng.integers(0, 200)), 1, j) for j in range(1, R + 1)] +
                        [(int(rng.integers(0, 300)), 0, int(j)) for j in rng.permutation(np.arange(1, R + 1))[: rng.integers(0, R)]])
        failed = set()
        for t, kind, j in events:
            if kind == 1:
                if j not in failed:
                    b.join(t, j)
            else:
                failed.add(j)
                b.fail(t, [j])
            _check_invariants(b)
        b.advance(10**7)
        _check_invariants(b)
        assert not b.waiting
        for r in b.locs[1:]:
            if r.alive:
                assert r.complete, (trial, r.obj)        # every live receiver ends with the whole object


def test_complete_copy_is_preferred_over_partial():
    b = BroadcastSchedule(0, 10, 1, 10)
    b.source_progress(0, 10)
    b.join(0, 1)          # S -> 1
    b.join(1, 2)          # 1 -> 2
    b.join(2, 3)          # 2 -> 3
    b.advance(105)        # 1 complete (t=100): S is free again
    b.join(105, 4)
    assert b.by_obj[4].first_sender_obj == 0


# ---------------------------------------------------------------- through the store: bytes
def test_store_broadcast_bytes_and_blocking_get():
    st = OracleStore(chunk_bytes=64, reduce_degree=2, bcast_degree=2, virt_chunk_ns=5)
    data = np.arange(100, dtype=np.float32)
    st.create(0, 0, 400, DT_F32)
    for j in range(1, 5):
        st.create(j, j, 400, DT_F32)
    st.put(0, data, 128)                 # two of seven chunks published
    st.broadcast(0, [1, 2, 3, 4])
    st.join(1)
    st.advance(3)
    st.join(2)
    with pytest.raises(StoreError) as ei:
        st.get(1)
    assert ei.value.code == ERR_TIMEOUT   # the source is still partial
    with pytest.raises(StoreError):
        st.get(3)                         # never joined
    st.advance(1000)
    st.put(0, data, 400)
    st.join(3)
    for j in (1, 2, 3):
        got = st.get(j)
        assert got.tobytes() == data.tobytes()
    w = st.dump(0)
    assert w[0] == 0x48504C42 and w[6] == 3


def test_a_rebuilt_receiver_holds_nothing_until_it_asks_again():
    """Section 3.5.1: a receiver whose worker failed and was rebuilt fetches the object again, as a new location.  Between
    the rebuild and that second request it holds no copy -- even if the copy it had before the failure was complete."""
    from oracle.store import OracleStore, StoreError, ERR_TIMEOUT, ERR_FAILED_WORKER, DT_F32
    st = OracleStore(64, 2, 1, 10)
    data = np.arange(64, dtype=np.float32)                 # 256 bytes = 4 chunks
    st.create(0, 9, 256, DT_F32)
    st.create(1, 1, 256, DT_F32)
    st.put(0, data, 256)
    st.broadcast(0, [1])
    st.join(1)
    assert st.get(1).tobytes() == data.tobytes()           # complete (the Get lets virtual time run)
    st.advance(st.now + 5)
    st.fail(1)
    with pytest.raises(StoreError) as ei:
        st.get(1)
    assert ei.value.code == ERR_FAILED_WORKER
    st.rejoin(1)
    with pytest.raises(StoreError) as ei:
        st.get(1)
    assert ei.value.code == ERR_TIMEOUT                    # rebuilt, not asked again
    st.join(1)
    assert st.get(1).tobytes() == data.tobytes()           # a new location, fetched again from the start
    assert [l.obj for l in st.bcasts[0]["sched"].locs] == [0, 1, 1]


def test_at_most_one_receiver_ever_waits():
    """Why the serving order among SEVERAL waiting receivers cannot be pinned: it cannot be observed.  A receiver waits only
    when no live location outside its own subtree has a free slot; a second receiver in that state could fetch from the
    first (a fresh receiver has all its slots), so two never wait at once -- checked here over random timelines in which
    the source, too, may fail, receivers fail in groups and are rebuilt."""
    rng = np.random.default_rng(47)
    most = 0
    for trial in range(600):
        C, d, tau, R = int(rng.integers(1, 10)), int(rng.integers(1, 4)), int(rng.integers(1, 20)), int(rng.integers(2, 14))
        b = BroadcastSchedule(0, C, d, tau)
        b.source_progress(0, int(rng.integers(0, C + 1)))
        t = 0
        alive = {j: True for j in range(0, R + 1)}
        for _ in range(int(rng.integers(R, 5 * R))):
            t += int(rng.integers(0, 3 * tau))
            r = rng.random()
            if r < 0.5:
                j = int(rng.integers(1, R + 1))
                if alive[j]:
                    b.join(t, j)
            elif r < 0.75:
                group = [int(x) for x in rng.choice(np.arange(0, R + 1), size=int(rng.integers(1, 4)), replace=False)]
                b.fail(t, group)
                for j in group:
                    alive[j] = False
            elif r < 0.85:
                j = int(rng.integers(1, R + 1))
                alive[j] = True                      # rebuilt: it may ask again (a new location)
            else:
                b.source_progress(t, C)
            most = max(most, len(b.waiting))
            assert len(b.waiting) <= 1, (trial, [w.obj for w in b.waiting])
    assert most == 1                                 # ... and one does wait in some of them
