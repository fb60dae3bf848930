"""Random timelines on the GPU: puts in instalments, failures, rejoins, joins, composed collectives and
explicit progress calls in random order, under random library flags.  Whenever the oracle can deliver an
object the library must deliver the same bits; whenever it cannot, the library must say the same."""
import numpy as np
import pytest
import torch

import paper_2002_05814_b200 as hpl
from oracle.store import StoreError, OK, DT_F32, DT_BF16
from tests.harness import Pair, gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2002_05814_b200 import build
    build.build()
    assert torch.cuda.is_available()


def _get_both(p: Pair, oid, plan_ahead):
    ro, want = OK, None
    try:
        want = p.o.get(oid)
    except StoreError as e:
        ro = e.code
    rl, ptr, n = p.c.try_get(oid)
    if plan_ahead and ro == OK and rl == hpl.HPL_ERR_TIMEOUT:
        p.c.sync()                                   # a polling kernel gave up earlier; its work is planned again
        rl, ptr, n = p.c.try_get(oid)
    assert rl == ro, (oid, ro, rl)
    if ro == OK:
        got = p.view(ptr, n).cpu().numpy().tobytes()
        assert got == want.tobytes(), f"object {oid} differs"
    if plan_ahead:
        p.c.sync()


def _timeline(seed, chunks=(4096, 16384)):
    rng = np.random.default_rng(seed)
    na, nb, R = int(rng.integers(2, 9)), int(rng.integers(1, 5)), int(rng.integers(1, 5))
    ka, kb = int(rng.integers(1, na + 1)), int(rng.integers(1, nb + 2))
    d = int(rng.integers(1, 5))
    chunk = int(rng.choice(list(chunks)))
    elems = int(rng.integers(1, 6)) * (chunk // 4) + int(rng.choice([0, 0, 3, 1000]))
    plan_ahead = bool(rng.random() < 0.3)
    flags = dict(fuse=bool(rng.random() < 0.6), eager=bool(rng.random() < 0.4), plan_ahead=plan_ahead,
                 poll_budget_ns=3_000_000 if plan_ahead else 0)
    p = Pair(chunk, d, int(rng.integers(1, 3)), tau=int(rng.integers(1, 50)), arena_bytes=32 << 20, **flags)
    arena_used_at_start = p.c.stats()["arena_used"]
    n = na + nb
    nbytes = elems * 4
    n_workers = max(1, int(rng.integers(1, n + 1)))
    a_bf16 = bool(rng.random() < 0.3)                 # the first Reduce takes bf16 inputs, its fp32 output feeds the second
    if a_bf16:
        elems -= elems % 8
    nbytes = elems * 4
    size_of = {}
    host_put = set()

    def put(i, nb_):
        if i in host_put:
            p.c.put_host(i, p.host[i].ctypes.data, nb_)
            p.o.put(i, p.host[i], nb_)
        else:
            p.put(i, nb_)

    for i in range(n):
        bf = a_bf16 and i < na
        data = gen(("normal", 0.02), 1000 + seed, i, elems, "bf16") if bf else \
            gen(("smallint", 30) if seed % 2 else ("uniform",), 1000 + seed, i, elems)
        size_of[i] = data.nbytes
        if rng.random() < 0.3:                        # this worker hands its object over from host memory
            host_put.add(i)
            p.host[i] = data
            wk = int(rng.integers(0, n_workers))
            p.c.create(i, wk, data.nbytes, DT_BF16 if bf else DT_F32)
            p.o.create(i, wk, data.nbytes, DT_BF16 if bf else DT_F32)
        else:
            p.create(i, int(rng.integers(0, n_workers)), data)
    for j in range(R):
        p.create(500 + j, 100 + int(rng.integers(0, 2)), nbytes=nbytes, dtype=DT_F32)
    A, B = 1000, 2000
    p.reduce(A, list(range(na)), ka, 0, DT_BF16 if a_bf16 else DT_F32)
    p.reduce(B, [A] + list(range(na, n)), kb)
    p.broadcast(B, [500 + j for j in range(R)])
    prefix = {i: 0 for i in range(n)}
    joiners = [500 + j for j in range(R)]
    t = 0
    for _ in range(int(rng.integers(2 * n, 6 * n + 8))):
        t = max(t + int(rng.integers(0, 40)), p.o.now)
        p.advance(t)
        r = rng.random()
        if r < 0.5:
            i = int(rng.integers(0, n))
            e = p.o.objects[i]
            if e.alive:
                nb_ = size_of[i] if rng.random() < 0.5 else min(size_of[i], prefix[i] + chunk)
                put(i, nb_)
                prefix[i] = nb_
        elif r < 0.6:
            p.fail(int(rng.integers(0, n_workers)))
        elif r < 0.66:
            wk = int(rng.integers(0, n_workers))
            p.c.rejoin(wk)
            p.o.rejoin(wk)
            for i in range(n):
                if p.o.objects[i].worker == wk and p.o.objects[i].alive and not p.o.objects[i].arrived:
                    prefix[i] = 0
        elif r < 0.76 and joiners:
            j = joiners.pop(0)
            if p.o.objects[j].alive:
                p.join(j)
        elif r < 0.86:
            p.progress()
        else:
            _get_both(p, int(rng.choice([A, B] + [500 + j for j in range(R)])), plan_ahead)
            t = max(t, p.o.now)
        for op in (A, B):
            p.check_schedule(op)
    for i in range(n):                                # let everything that is still alive complete
        if p.o.objects[i].alive:
            t = max(t + 5, p.o.now)
            p.advance(t)
            put(i, size_of[i])
    for oid in [A, B] + [500 + j for j in range(R)]:
        _get_both(p, oid, plan_ahead)
    p.check_schedule(A)
    p.check_schedule(B)
    if plan_ahead:
        p.c.sync()
    for oid in [B, A] + list(range(n)):               # consumers before what they consume; receivers go with their broadcast
        p.delete(oid)
    assert p.c.stats()["arena_used"] == arena_used_at_start, "arena blocks are left after every object was deleted"
    p.close()


@pytest.mark.parametrize("block", range(8))
def test_random_timelines_match_the_oracle(block):
    for seed in range(block * 40, (block + 1) * 40):
        try:
            _timeline(seed)
        except AssertionError as e:
            raise AssertionError(f"seed {seed}: {e}") from e


@pytest.mark.parametrize("block", range(3))
def test_random_timelines_with_objects_above_the_small_object_threshold(block):
    """The same timelines with chunks of 32 and 64 KiB: objects of 32 KiB to 320 KiB, most of them above the 64 KiB
    under which collectives share their waves."""
    for seed in range(5000 + block * 40, 5000 + (block + 1) * 40):
        try:
            _timeline(seed, chunks=(32768, 65536))
        except AssertionError as e:
            raise AssertionError(f"seed {seed}: {e}") from e


@pytest.mark.parametrize("seed", [639, 1088, 1166, 1199, 1221, 1471])
def test_small_collectives_beside_a_polling_one_whose_wait_runs_out(seed):
    """Timelines in which a small collective (its tasks wait for a shared wave) is planned in the same pass as one whose
    polling wave gives up: the wait that ran out must void exactly the pass that launched it and the later ones -- not
    the small collective planned before it, whose wave completed -- and must void all of its own pass."""
    _timeline(seed)


def _tight_arena_timeline(seed):
    """Several Reduces whose tree nodes keep their reduced objects, in an arena that holds the outputs and only a few
    partial results: buffers are evicted and made again all the time.  Returns the number of evictions, or None when
    even the pinned copies did not fit."""
    rng = np.random.default_rng(seed)
    n_ops = int(rng.integers(2, 6))
    chunk = int(rng.choice([4096, 16384, 65536]))
    elems = int(rng.integers(1, 5)) * (chunk // 4) + int(rng.choice([0, 3]))
    S = elems * 4
    fixed = 4096 * 32 + 256 * 32 + (64 << 10)
    ks = [int(rng.integers(2, 9)) for _ in range(n_ops)]
    room = n_ops + int(rng.integers(1, 6))                  # the outputs are pinned; a few more buffers for partial results
    p = Pair(chunk, int(rng.integers(1, 4)), fuse=bool(rng.random() < 0.3), eager=bool(rng.random() < 0.3),
             arena_bytes=fixed + room * (((S + 255) // 256) * 256 + 512))
    oid, ops = 0, []
    for q in range(n_ops):
        ids = list(range(oid, oid + ks[q] + 1))
        oid += ks[q] + 1
        for i in ids:
            p.create(i, i, gen(("smallint", 20) if seed % 2 else ("uniform",), 700 + seed, i, elems))
        ops.append((1000 + q, ids))

    def check(tgt, final):
        ro, want = OK, None
        try:
            want = p.o.get(tgt)
        except StoreError as e:
            ro = e.code
        rl, ptr, nb = p.c.try_get(tgt)
        if rl == hpl.HPL_ERR_NOMEM:
            raise hpl.HplError(rl, "hpl_get")
        assert rl == ro, (tgt, ro, rl)
        if ro == OK:
            assert p.view(ptr, nb).cpu().numpy().tobytes() == want.tobytes(), f"target {tgt} differs"
            if final:
                p.check_schedule(tgt)

    def tolerant(call, *a):
        """The library's half of an event whose planning may run out of arena: the event itself is applied all the same
        (the oracle's half follows), only the work it would have started is not."""
        try:
            call(*a)
        except hpl.HplError as e:
            if e.code != hpl.HPL_ERR_NOMEM:
                raise
            nomem[0] += 1

    nomem = [0]
    try:
        for tgt, ids in ops:
            p.reduce(tgt, ids, len(ids) - 1)                # one spare each
    except hpl.HplError as e:                               # not even the outputs fit
        if e.code != hpl.HPL_ERR_NOMEM:
            raise
        p.c.shutdown()
        return None
    pend = [i for _, ids in ops for i in ids]
    t = 0
    for idx in rng.permutation(len(pend)):
        i = pend[idx]
        t += int(rng.integers(0, 10))
        p.advance(t)
        if rng.random() < 0.85:
            nb_ = S if rng.random() < 0.7 else min(S, chunk)
            tolerant(p.c.put, i, p.dev[i].data_ptr(), nb_)
            p.o.put(i, p.host[i], nb_)
        r = rng.random()
        if r < 0.3:
            tolerant(p.progress)
        elif r < 0.38 and p.o.objects[i].alive:
            tolerant(p.c.fail, i)
            p.o.fail(i)
        elif r < 0.5:
            tolerant(check, ops[int(rng.integers(0, n_ops))][0], False)
    for _, ids in ops:
        for i in ids:
            if p.o.objects[i].alive:
                t += 1
                p.advance(t)
                tolerant(p.c.put, i, p.dev[i].data_ptr(), S)
                p.o.put(i, p.host[i], S)
    done = []
    for tgt, ids in ops:
        try:
            check(tgt, True)
        except hpl.HplError as e:
            if e.code != hpl.HPL_ERR_NOMEM:
                raise
            # a pass that ran out of arena left nothing half done: make room (the outputs checked so far go, with their
            # partial results) and ask again
            nomem[0] += 1
            for d_tgt, d_ids in done:
                p.delete(d_tgt)
                for i in d_ids:
                    p.delete(i)
            done = []
            try:
                check(tgt, True)
            except hpl.HplError as e2:
                if e2.code != hpl.HPL_ERR_NOMEM:
                    raise
                p.c.shutdown()
                return None
        done.append((tgt, ids))
    ev = p.c.stats()["evictions"]
    p.close()
    return ev


def test_random_timelines_in_arenas_too_small_for_all_partial_results():
    evictions = 0
    for seed in range(120):
        try:
            evictions += _tight_arena_timeline(seed) or 0
        except AssertionError as e:
            raise AssertionError(f"seed {seed}: {e}") from e
    assert evictions > 50
