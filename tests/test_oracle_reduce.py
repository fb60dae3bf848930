"""Pins for the reduce half of the oracle: the paper's worked example, closed forms, special
cases that reduce to a plain left-to-right sum, invariants and brute force on tiny inputs."""
import itertools
import math

import numpy as np
import pytest

from oracle import reduce_tree as rt
from oracle import values as ov
from oracle.store import OracleStore, StoreError, ERR_TIMEOUT, ERR_INSUFFICIENT, DT_F32, DT_BF16
from tests.conftest import read_golden


def _bits(words):
    return np.array([int(w, 16) for w in words.split()], dtype=np.uint32).view(np.float32)


def _read_inorder(obj_at, d):
    """Independent reading of a finished tree: recursive, straight from the sentence in Section 3.4.2."""
    k = len(obj_at)

    def kids(p):
        return [c for c in range(d * p + 1, d * p + d + 1) if c < k]

    def walk(p):
        ks = kids(p)
        first = walk(ks[0]) if ks else []
        rest = [x for c in ks[1:] for x in walk(c)]
        return first + [obj_at[p]] + rest

    return walk(0)


def _build(k, d, n=None, order=None):
    n = n or k
    s = rt.ReduceSchedule(list(range(n)), k, d)
    for o in (order or range(n)):
        s.on_arrival(o)
    return s


# ---------------------------------------------------------------- worked example (Fig. 5, text)
def test_paper_example_six_objects_binary():
    g = read_golden("reduce_example_6_binary.txt")
    names = g["arrival_order"].split()
    s = _build(6, 2)
    read = [names[o] for o in _read_inorder(s.obj_at, 2)]
    assert read == g["inorder_reads"].split()
    # R4 is an ancestor of R2, and the root
    p2, p4 = s.pos_of[names.index("R2")], s.pos_of[names.index("R4")]
    assert p4 in rt.ancestors(p2, 2) and p4 == 0


def test_paper_example_failure_r2_replaced_by_r7():
    g = read_golden("reduce_example_6_binary.txt")
    name = lambda o: f"R{o + 1}"
    for r7_before_failure in (True, False):
        s = rt.ReduceSchedule(list(range(10)), 6, 2)
        for o in range(6):
            s.on_arrival(o)
        pos_r2 = s.pos_of[1]
        if r7_before_failure:
            s.on_arrival(6)
        s.on_fail(1, 3)
        if not r7_before_failure:
            assert not s.full()
            s.on_arrival(6)
        assert s.full()
        assert sorted(name(o) for o in s.members()) == sorted(g["final_members"].split())
        assert s.pos_of[6] == pos_r2                       # R7 takes R2's position
        cleared = [name(s.obj_at[p]) for p in s.edits[-1].cleared]
        assert cleared == g["clears"].split()               # only R4 clears
        assert len(s.edits[-1].cleared) <= math.ceil(math.log(6, 2))


def test_hand_worked_association_bits():
    g = read_golden("reduce_association_bits.txt")
    for key, k in (("k3", 3), ("k6", 6)):
        x = _bits(g[f"{key}_inputs"])
        s = _build(k, 2)
        objs = {i: np.array([x[i]], dtype=np.float32) for i in range(k)}
        got = ov.tree_reduce(s.obj_at, 2, objs)
        assert got.view(np.uint32)[0] == int(g[f"{key}_result"], 16)
    chain = ov.naive_reduce_f32(list(range(6)), {i: np.array([_bits(g["k6_inputs"])[i]], dtype=np.float32) for i in range(6)})
    assert chain.view(np.uint32)[0] == int(g["k6_chain_result"], 16)


# ---------------------------------------------------------------- shape: invariants and special cases
@pytest.mark.parametrize("d", [1, 2, 3, 4, 7, 64])
@pytest.mark.parametrize("k", [1, 2, 3, 5, 6, 8, 13, 32, 64])
def test_inorder_is_a_permutation_and_reads_back_in_arrival_order(k, d):
    order = rt.inorder(k, d)
    assert sorted(order) == list(range(k))
    s = _build(k, d)
    assert _read_inorder(s.obj_at, d) == list(range(k))      # arrival i sits at in-order rank i
    assert sorted(s.members()) == list(range(k))             # each object exactly once
    # every non-root has its parent inside the tree, degree <= d
    for p in range(1, k):
        assert 0 <= rt.parent(p, d) < p
    assert all(len(rt.children(p, d, k)) <= d for p in range(k))
    if d >= 2:
        height = max(len(rt.ancestors(p, d)) for p in range(k))
        assert height == math.ceil(math.log(k * (d - 1) + 1, d) - 1e-9) - 1


def test_chain_and_star_are_left_to_right_sums():
    rng = np.random.default_rng(5)
    k = 9
    objs = {i: rng.uniform(-1, 1, 257).astype(np.float32) for i in range(k)}
    arrival = [4, 0, 8, 2, 6, 1, 7, 3, 5]
    want = ov.naive_reduce_f32(arrival, objs)
    for d in (1, k - 1, k, 50):      # d = 1: the chain of Eq. 1; d >= k-1: the star
        s = _build(k, d, order=arrival)
        got = ov.tree_reduce(s.obj_at, d, objs)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), d
    s = _build(k, 1, order=arrival)
    assert [s.obj_at[p] for p in range(k)] == arrival[::-1]   # first arrival is the far end of the chain
    s = _build(k, k, order=arrival)
    assert s.obj_at[0] == arrival[1] and rt.children(0, k, k) == list(range(1, k))


@pytest.mark.parametrize("d", [1, 2, 3, 4])
def test_k_of_m_takes_the_earliest_arrivals(d):
    n = 10
    for k in range(1, n + 1):
        arrival = list(np.random.default_rng(k).permutation(n))
        s = _build(k, d, n=n, order=arrival)
        assert set(s.members()) == set(arrival[:k])
        assert s.spares == arrival[k:]


# ---------------------------------------------------------------- values: brute force
@pytest.mark.parametrize("d", [1, 2, 3, 4, 8])
def test_integer_inputs_equal_brute_force_bit_for_bit(d):
    rng = np.random.default_rng(11)
    for k in (1, 2, 5, 8, 10):
        objs = {i: rng.integers(-1000, 1000, 64).astype(np.float32) for i in range(k)}
        s = _build(k, d)
        got = ov.tree_reduce(s.obj_at, d, objs)
        want = ov.naive_sum_f64(list(range(k)), objs)
        assert np.array_equal(got.astype(np.float64), want)
        for op, fn in ((ov.OP_MIN, np.minimum), (ov.OP_MAX, np.maximum)):
            ref = objs[0]
            for i in range(1, k):
                ref = fn(ref, objs[i])
            assert np.array_equal(ov.tree_reduce(s.obj_at, d, objs, op), ref)


@pytest.mark.parametrize("k,d", [(8, 2), (64, 4), (32, 2), (16, 1)])
def test_fp32_tree_within_bound_of_fp64_sum(k, d):
    rng = np.random.default_rng(3)
    objs = {i: rng.uniform(-1, 1, 4096).astype(np.float32) for i in range(k)}
    s = _build(k, d)
    got = ov.tree_reduce(s.obj_at, d, objs).astype(np.float64)
    ref = ov.naive_sum_f64(list(range(k)), objs)
    err = np.max(np.abs(got - ref)) / np.max(np.abs(ref))
    assert err <= 1e-5 * math.ceil(math.log2(k))


def test_bf16_inputs_are_widened_exactly():
    import torch
    rng = np.random.default_rng(2)
    f = rng.normal(0, 0.02, 1000).astype(np.float32)
    t = torch.from_numpy(f).to(torch.bfloat16)
    u16 = t.view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ov.widen(u16), t.to(torch.float32).numpy())


# ---------------------------------------------------------------- failures: every position, several times
def _expected_members(arrival, failed, k):
    live = [o for o in arrival if o not in failed]
    return set(live[:k])


@pytest.mark.parametrize("d", [1, 2, 3, 4])
def test_single_failure_everywhere_matches_survivor_sum(d):
    rng = np.random.default_rng(17)
    n = 7
    objs = {i: rng.integers(-50, 50, 16).astype(np.float32) for i in range(n)}
    for k in (3, 5, 7):
        for victim in range(n):
            for when in range(n + 1):          # the failure comes after `when` arrivals
                s = rt.ReduceSchedule(list(range(n)), k, d)
                for i in range(n):
                    if i == when:
                        s.on_fail(victim, 2, lambda o: 4)
                    if not (i == victim and when <= i):
                        s.on_arrival(i)
                if when == n:
                    s.on_fail(victim, 2, lambda o: 4)
                k_eff = min(k, n - 1)
                assert s.k == k_eff and s.full()
                members = s.members()
                assert len(set(members)) == k_eff and victim not in members
                arrival = [i for i in range(n) if not (i == victim and when <= i)]
                assert set(members) == _expected_members(arrival, {victim}, k_eff)
                got = ov.tree_reduce(s.obj_at, d, objs)
                assert np.array_equal(got.astype(np.float64), ov.naive_sum_f64(members, objs))
                for e in s.edits:              # Section 3.5.2: only ancestors clear, at most two root paths
                    bound = math.ceil(math.log(max(k, 2), max(d, 2))) if d > 1 else k
                    assert len(e.cleared) <= (2 if e.kind == rt.EDIT_SHRINK else 1) * max(bound, 1)
                    for c in e.cleared:
                        assert 0 <= c < k


def test_random_failure_sequences_keep_invariants():
    rng = np.random.default_rng(23)
    for trial in range(300):
        n = int(rng.integers(2, 12))
        k = int(rng.integers(1, n + 1))
        d = int(rng.integers(1, 5))
        s = rt.ReduceSchedule(list(range(n)), k, d)
        events = [("a", o) for o in rng.permutation(n)] + [("f", o) for o in rng.permutation(n)[: rng.integers(0, n)]]
        events = [events[i] for i in rng.permutation(len(events))]
        arrived, failed = [], set()
        for kind, o in events:
            if kind == "a":
                if o not in failed:
                    arrived.append(o)
                s.on_arrival(o)
            else:
                failed.add(o)
                s.on_fail(o, 1, lambda x: 1)
            assert s.live_count() >= s.k
            m = s.members()
            assert len(m) == len(set(m)) and not (set(m) & failed)
            assert all(s.obj_at[s.pos_of[x]] == x for x in m)
        live_arrived = [o for o in arrived if o not in failed]
        assert s.k == min(k, n - len(failed))
        assert set(s.members()) == set(live_arrived[: s.k]) or len(live_arrived) < s.k


# ---------------------------------------------------------------- the store: timeline semantics
def _store_with(n, k, d, elems=64, dtype=DT_F32):
    st = OracleStore(chunk_bytes=64, reduce_degree=d, bcast_degree=1)
    rng = np.random.default_rng(1)
    data = {}
    for i in range(n):
        st.create(i, i, elems * 4, dtype)
        data[i] = rng.integers(-9, 9, elems).astype(np.float32)
    return st, data


def test_store_reduce_first_k_ready_and_blocking():
    st, data = _store_with(6, 3, 2)
    st.reduce(100, list(range(6)), 3)
    with pytest.raises(StoreError) as ei:
        st.get(100)
    assert ei.value.code == ERR_TIMEOUT
    for t, o in ((10, 4), (20, 1), (30, 5), (40, 0)):
        st.advance(t)
        st.put(o, data[o], data[o].nbytes if o != 5 else 128)    # object 5 arrives partial
    with pytest.raises(StoreError):
        st.get(100)                                              # 5 is selected but incomplete
    st.advance(50)
    st.put(5, data[5], data[5].nbytes)
    got = st.get(100)
    assert np.array_equal(got, data[4] + data[1] + data[5])      # the first three to arrive


def test_store_failure_without_spare_sums_the_survivors():
    st, data = _store_with(5, 5, 2)
    for o in range(5):
        st.put(o, data[o], data[o].nbytes if o != 2 else 64)
    st.reduce(100, list(range(5)), 5)
    st.advance(5)
    st.fail(2)
    got = st.get(100)
    assert np.array_equal(got, sum(data[o] for o in (0, 1, 3, 4)))
    w = st.dump(100)
    assert w[0] == 0x48504C52 and w[3] == 5 and w[4] == 4


def test_store_reduce_with_no_live_source_is_insufficient():
    st, data = _store_with(3, 2, 2)
    st.reduce(100, [0, 1, 2], 2)
    st.put(0, data[0], data[0].nbytes)
    for w in (0, 1, 2):
        st.fail(w)
    with pytest.raises(StoreError) as ei:
        st.get(100)
    assert ei.value.code == ERR_INSUFFICIENT


# ---------------------------------------------------------------- composition (Sections 3.3, 3.4.2, 3.4.3)
def test_composed_reduce_and_allreduce_equal_the_plain_sums():
    st, data = _store_with(6, 3, 2, elems=64)
    st.reduce(100, [0, 1, 2], 3)                 # first Reduce: a future
    st.reduce(200, [100, 3, 4], 3)               # its output id is an input of the next one
    for j in (300, 301, 302):
        st.create(j, 50 + j, 256, DT_F32)
    st.broadcast(200, [300, 301, 302])           # reduce followed by broadcast = allreduce
    st.join(300)
    with pytest.raises(StoreError):
        st.get(200)
    st.advance(1)
    for o in (0, 1):
        st.put(o, data[o], 256)
    st.put(2, data[2], 128)                      # object 2 is half there: so is the first output
    assert st._delivered(100) == 2 and st._delivered(200) == 0
    st.advance(2)
    for o in (3, 4):
        st.put(o, data[o], 256)
    assert st._delivered(200) == 2               # the partial first output already feeds the second Reduce
    st.join(301)
    st.advance(3)
    st.put(2, data[2], 256)
    st.join(302)
    total = sum(data[o] for o in range(5))       # integer-valued inputs: any association is exact
    assert np.array_equal(st.get(100), data[0] + data[1] + data[2])
    assert np.array_equal(st.get(200), total)
    for j in (300, 301, 302):
        assert st.get(j).tobytes() == total.astype(np.float32).tobytes()
    # each input was reduced once and only once (Section 3.4.2)
    ones = {o: np.ones(64, np.float32) for o in range(5)}
    st2, _ = _store_with(6, 3, 2, elems=64)
    st2.reduce(100, [0, 1, 2], 3)
    st2.reduce(200, [100, 3, 4], 3)
    for o in range(5):
        st2.put(o, ones[o], 256)
    assert np.array_equal(st2.get(200), np.full(64, 5, np.float32))


def test_composed_reduce_redoes_the_downstream_after_an_upstream_failure():
    st, data = _store_with(6, 3, 2, elems=64)
    st.reduce(100, [0, 1, 2, 5], 3)
    st.reduce(200, [100, 3], 2)
    for o in (0, 1, 2, 3):
        st.put(o, data[o], 256)
    assert np.array_equal(st.get(200), data[0] + data[1] + data[2] + data[3])
    st.advance(9)
    st.fail(1)                                   # a member of the first Reduce is lost; object 5 is its spare
    with pytest.raises(StoreError):
        st.get(200)
    st.put(5, data[5], 256)
    assert np.array_equal(st.get(200), data[0] + data[5] + data[2] + data[3])


# ---------------------------------------------------------------- rejoin (Section 3.5) and degree choice (Eq. 1)
def test_rejoined_source_counts_as_a_new_arrival():
    # "R7 can also be the rejoined R2": reduce 6 of 6, R2 fails, is rebuilt and put again
    s = rt.ReduceSchedule(list(range(6)), 6, 2)
    for o in range(6):
        s.on_arrival(o)
    pos = s.pos_of[1]
    s.on_fail(1, 2, lambda o: 4)
    assert s.k == 5                                   # no spare: the tree shrank (build-defined)
    s.on_rejoin(1)
    s.on_arrival(1)
    assert s.spares == [1] and s.live_count() == 6    # it does not grow back; the source waits as a spare
    s2 = rt.ReduceSchedule(list(range(7)), 6, 2)      # with a seventh source still to come the position stays open
    for o in range(6):
        s2.on_arrival(o)
    s2.on_fail(1, 2, lambda o: 4)
    assert not s2.full() and s2.k == 6
    s2.on_rejoin(1)
    s2.on_arrival(1)
    assert s2.full() and s2.pos_of[1] == pos          # the rebuilt R2 takes its old position back
    st, data = _store_with(4, 3, 2)
    st.reduce(100, [0, 1, 2, 3], 4)
    for o in range(4):
        st.put(o, data[o], 256)
    st.fail(2)
    assert np.array_equal(st.get(100), data[0] + data[1] + data[3])
    st.rejoin(2)
    with pytest.raises(StoreError) as ei:
        st.get(2)
    assert ei.value.code == ERR_TIMEOUT               # a future again
    st.put(2, data[2], 256)
    assert np.array_equal(st.get(100), data[0] + data[1] + data[3])   # the shrunk tree is complete without it


def test_degree_choice_follows_eq_1():
    L, B = 100e-6, 1.25e9                             # 100 us, 10 Gbit/s
    # the three closed forms of Section 3.4.2
    for n in (2, 4, 8, 16):
        for S in (1e3, 1e6, 1e9):
            t = {1: n * L + S / B, 2: L * math.log2(n) + 2 * S / B, n: L + n * S / B}
            want = min(sorted(t), key=lambda d: (t[d], d))
            assert rt.choose_degree(n, S, L, B) == want
    assert rt.choose_degree(16, 1e3, L, B) == 16      # small objects: latency dominates, d = n
    assert rt.choose_degree(16, 1e9, L, B) == 1       # large objects: bandwidth dominates, the chain
    assert rt.choose_degree(16, 4e5, L, B) == 2       # in between
    assert rt.choose_degree(1, 1e6, L, B) == 1
