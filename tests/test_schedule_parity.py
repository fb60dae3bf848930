"""Schedules built by the library (host code, no GPU needed) against the oracle, bit for bit, on
randomised timelines of puts, joins, failures and gets."""
import numpy as np
import pytest

import paper_2002_05814_b200 as hpl
from oracle.store import OracleStore, StoreError, OK, ERR_TIMEOUT
from paper_2002_05814_b200 import build as hpl_build


@pytest.fixture(scope="module", autouse=True)
def _built():
    hpl_build.build()


CHUNK = 64


class Pair:
    """Drives the oracle and a schedule-only library context with the same events."""

    def __init__(self, d_reduce, d_bcast, tau):
        self.o = OracleStore(CHUNK, d_reduce, d_bcast, tau)
        self.c = hpl.Context(CHUNK, d_reduce, d_bcast, virt_chunk_ns=tau)
        self.data = {}
        self.addr = {}

    def close(self):
        self.c.shutdown()

    def both(self, name, *args, oracle_args=None):
        ro = OK
        try:
            getattr(self.o, name)(*(oracle_args if oracle_args is not None else args))
        except StoreError as e:
            ro = e.code
        rl = OK
        try:
            getattr(self.c, name)(*args)
        except hpl.HplError as e:
            rl = e.code
        assert ro == rl, (name, args, ro, rl)
        return ro

    def create(self, oid, worker, nbytes):
        self.data[oid] = np.zeros(nbytes // 4, np.float32)
        self.addr[oid] = 4096 * (oid + 1)
        return self.both("create", oid, worker, nbytes, 0)

    def put(self, oid, nbytes):
        ro = OK
        try:
            self.o.put(oid, self.data[oid], nbytes)
        except StoreError as e:
            ro = e.code
        rl = OK
        try:
            self.c.put(oid, self.addr[oid], nbytes)
        except hpl.HplError as e:
            rl = e.code
        assert ro == rl, ("put", oid, nbytes, ro, rl)

    def join(self, oid):
        ro = OK
        try:
            self.o.join(oid)
        except StoreError as e:
            ro = e.code
        rl = OK
        try:
            self.c.join(oid, None)
        except hpl.HplError as e:
            rl = e.code
        assert ro == rl, ("join", oid, ro, rl)

    def get(self, oid):
        ro = OK
        try:
            self.o.get(oid)
        except StoreError as e:
            ro = e.code
        rl, _, _ = self.c.try_get(oid)
        if ro == OK:
            assert rl == hpl.HPL_ERR_CUDA, (oid, rl)   # would succeed with a device
        else:
            assert rl == ro, ("get", oid, ro, rl)
        return ro

    def compare(self, op_id):
        assert self.c.schedule_dump(op_id) == self.o.dump(op_id)


def _reduce_timeline(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 13))
    k = int(rng.integers(1, n + 1))
    d = int(rng.integers(1, 5))
    nbytes = int(rng.integers(1, 9)) * 64 - (0 if rng.random() < 0.7 else 60)
    p = Pair(d, 1, 7)
    n_workers = max(1, int(rng.integers(1, n + 1)))
    for i in range(n):
        p.create(i, int(rng.integers(0, n_workers)), nbytes)
    t = 0
    called = False
    order = list(rng.permutation(n))
    prefix = {i: 0 for i in range(n)}
    steps = int(rng.integers(n, 4 * n + 4))
    for s in range(steps):
        t += int(rng.integers(0, 20))
        p.both("advance", t)
        r = rng.random()
        if not called and (r < 0.25 or s == steps // 2):
            if p.both("reduce", 1000, list(range(n)), k, 0, 0) != OK:
                p.close()
                return        # refused alike by both (e.g. no live source left)
            called = True
        elif r < 0.7 and order:
            i = int(order[0])
            full = rng.random() < 0.6
            nb = nbytes if full else int(rng.integers(prefix[i], nbytes + 1))
            nb -= nb % 4
            nb = max(nb, prefix[i])
            if nb == 0:
                nb = nbytes
            p.put(i, nb)
            prefix[i] = nb
            if nb == nbytes:
                order.pop(0)
        elif r < 0.82:
            p.both("fail", int(rng.integers(0, n_workers)))
        elif r < 0.88:
            wk = int(rng.integers(0, n_workers))
            p.both("rejoin", wk)
            for i in range(n):                      # a rebuilt worker's objects are futures again
                if p.o.objects[i].worker == wk and p.o.objects[i].alive and not p.o.objects[i].arrived:
                    prefix[i] = 0
                    if i not in order:
                        order.append(i)
        elif called:
            p.get(1000)
        if called:
            p.compare(1000)
    if called:
        p.get(1000)
        p.compare(1000)
    p.close()


@pytest.mark.parametrize("block", range(8))
def test_reduce_schedules_match_on_random_timelines(block):
    for seed in range(block * 150, (block + 1) * 150):
        _reduce_timeline(seed)


def _bcast_timeline(seed, complete_source=False):
    rng = np.random.default_rng(seed)
    R = int(rng.integers(1, 14))
    d = int(rng.integers(1, 4))
    tau = int(rng.integers(1, 30))
    nbytes = int(rng.integers(1, 12)) * 64
    p = Pair(2, d, tau)
    n_workers = int(rng.integers(1, R + 2))
    p.create(0, int(rng.integers(0, n_workers)) if rng.random() < 0.3 else 99, nbytes)
    for j in range(1, R + 1):
        p.create(j, int(rng.integers(0, n_workers)), nbytes)
    t = 0
    src_pref = 0
    if rng.random() < 0.5 or complete_source:
        src_pref = nbytes if (rng.random() < 0.6 or complete_source) else int(rng.integers(0, nbytes // 64 + 1)) * 64
        if src_pref:
            p.put(0, src_pref)
    p.both("broadcast", 0, list(range(1, R + 1)))
    joiners = list(rng.permutation(np.arange(1, R + 1)))
    for s in range(int(rng.integers(R, 4 * R + 6))):
        t += int(rng.integers(0, 3 * tau))
        p.both("advance", t)
        t = max(t, p.o.now)
        r = rng.random()
        if r < 0.45 and joiners:
            p.join(int(joiners.pop(0)))
        elif r < 0.6 and src_pref < nbytes:
            src_pref = nbytes if rng.random() < 0.5 else min(nbytes, src_pref + 64)
            p.put(0, src_pref)
        elif r < 0.72:
            p.both("fail", int(rng.integers(0, n_workers)))
        elif r < 0.8:
            wk = int(rng.integers(0, n_workers))
            p.both("rejoin", wk)
            for j in range(1, R + 1):               # rebuilt receivers ask again
                if p.o.objects[j].worker == wk and j not in joiners and rng.random() < 0.7:
                    joiners.append(j)
        else:
            p.get(int(rng.integers(1, R + 1)))
            t = max(t, p.o.now)
        p.compare(0)
    if src_pref < nbytes:
        p.put(0, nbytes)
    for j in range(1, R + 1):
        p.get(j)
        p.compare(0)
    p.close()


@pytest.mark.parametrize("block", range(8))
def test_broadcast_schedules_match_on_random_timelines(block):
    for seed in range(block * 150, (block + 1) * 150):
        _bcast_timeline(seed)


@pytest.mark.parametrize("block", range(4))
def test_broadcasts_of_a_complete_source_match_through_failures(block):
    """The library computes these in closed form (evenly spaced landings) until something fails or waits, then goes
    on chunk by chunk; the oracle simulates every chunk throughout."""
    for seed in range(10_000 + block * 150, 10_000 + (block + 1) * 150):
        _bcast_timeline(seed, complete_source=True)


def _composed_timeline(seed):
    """Reduce A, Reduce B that takes A's output as an input, and a broadcast of B's output (allreduce)."""
    rng = np.random.default_rng(seed)
    na, nb, R = int(rng.integers(1, 6)), int(rng.integers(1, 5)), int(rng.integers(1, 6))
    ka = int(rng.integers(1, na + 1))
    kb = int(rng.integers(1, nb + 2))
    d = int(rng.integers(1, 4))
    tau = int(rng.integers(1, 20))
    nbytes = int(rng.integers(1, 6)) * 64
    p = Pair(d, int(rng.integers(1, 3)), tau)
    n = na + nb
    n_workers = max(1, int(rng.integers(1, n + 1)))
    for i in range(n):
        p.create(i, int(rng.integers(0, n_workers)), nbytes)
    for j in range(R):
        p.create(500 + j, 100 + int(rng.integers(0, 3)), nbytes)
    A, B = 1000, 2000
    ops = []
    if p.both("reduce", A, list(range(na)), ka, 0, 0) != OK:
        p.close()
        return
    ops.append(A)
    if p.both("reduce", B, [A] + list(range(na, n)), kb, 0, 0) == OK:
        ops.append(B)
        if p.both("broadcast", B, [500 + j for j in range(R)]) == OK:
            ops.append("bcast")
    prefix = {i: 0 for i in range(n)}
    joiners = [500 + j for j in range(R)]
    t = 0
    for s in range(int(rng.integers(n, 5 * n + 6))):
        t += int(rng.integers(0, 2 * tau))
        p.both("advance", max(t, p.o.now))
        t = max(t, p.o.now)
        r = rng.random()
        if r < 0.5:
            i = int(rng.integers(0, n))
            nb_ = nbytes if rng.random() < 0.5 else min(nbytes, prefix[i] + 64)
            p.put(i, nb_)
            if p.o.objects[i].alive:
                prefix[i] = max(prefix[i], nb_)
        elif r < 0.62:
            p.both("fail", int(rng.integers(0, n_workers)))
        elif r < 0.8 and joiners and "bcast" in ops:
            p.join(joiners.pop(0))
        else:
            p.get(int(rng.choice([A, B] + [500 + j for j in range(R)])) if len(ops) > 1 else A)
            t = max(t, p.o.now)
        for o in ops:
            p.compare(B if o == "bcast" else o)
    p.close()


@pytest.mark.parametrize("block", range(4))
def test_composed_schedules_match_on_random_timelines(block):
    for seed in range(block * 150, (block + 1) * 150):
        _composed_timeline(seed)


def test_degree_choice_matches_the_oracle():
    from oracle.reduce_tree import choose_degree
    rng = np.random.default_rng(9)
    for _ in range(3000):
        n = int(rng.integers(1, 200))
        S = int(10 ** rng.uniform(1, 10))
        L = float(10 ** rng.uniform(-7, -2))
        B = float(10 ** rng.uniform(8, 12))
        assert hpl.choose_degree(n, S, L, B) == choose_degree(n, float(S), L, B)
    # through the store: degree 0 means "choose per Reduce"
    for nbytes, want in ((64, 4), (64 * 4096, 1)):
        o = OracleStore(64, 0, 1, 0, model_latency_ns=1000, model_bandwidth_bps=10**9)
        c = hpl.Context(64, 0, 1, model_latency_ns=1000, model_bandwidth_bps=10**9)
        for i in range(4):
            o.create(i, i, nbytes, 0)
            c.create(i, i, nbytes)
        o.reduce(100, [0, 1, 2, 3], 4)
        c.reduce(100, [0, 1, 2, 3], 4)
        assert c.schedule_dump(100) == o.dump(100) and o.dump(100)[5] == want
        c.shutdown()
