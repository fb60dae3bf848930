"""Parity of the CUDA broadcast path with the oracle (through the C ABI), byte by byte."""
import numpy as np
import pytest
import torch

import paper_2002_05814_b200 as hpl
import workloads as wl
from oracle.store import StoreError, OK, DT_F32, DT_BF16
from tests.harness import Pair, gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2002_05814_b200 import build
    build.build()
    assert torch.cuda.is_available()


@pytest.mark.parametrize("nbytes,chunk,R,d,dtype", [
    (1 << 20, 64 << 10, 16, 2, "f32"), (4 * 30_001, 16 << 10, 5, 1, "f32"), (2 * 50_001, 16 << 10, 7, 3, "bf16"),
    (2 * 7, 4096, 3, 2, "bf16"), (1 << 16, 1 << 20, 64, 4, "f32"),
])
def test_staggered_joins_every_receiver_gets_the_bytes(nbytes, chunk, R, d, dtype):
    elems = nbytes // (4 if dtype == "f32" else 2)
    p = Pair(chunk, 2, d)
    p.create(0, 99, gen(("uniform",), 31, 0, elems, dtype))
    for j in range(1, R + 1):
        p.create(j, j, nbytes=nbytes, dtype=DT_F32 if dtype == "f32" else DT_BF16)
    p.put(0)
    p.broadcast(0, list(range(1, R + 1)))
    joins = sorted((t, j + 1) for j, t in enumerate(wl.uniform_offsets_ns(5, R)))
    for n, (t, j) in enumerate(joins):
        p.advance(t)
        p.join(j)
        if n % 3 == 2:
            p.progress()           # some receivers are served early, later ones read from their senders' copies
    p.check_schedule(0)
    for j in range(1, R + 1):
        p.check_receiver_bytes(j)
    p.check_schedule(0)
    p.close()


def test_all_join_before_any_launch_is_one_read_many_writes():
    nbytes, R = 1 << 20, 16
    p = Pair(64 << 10, 2, 2)
    p.create(0, 99, gen(("uniform",), 1, 0, nbytes // 4))
    for j in range(1, R + 1):
        p.create(j, j, nbytes=nbytes, dtype=DT_F32)
    p.put(0)
    p.broadcast(0, list(range(1, R + 1)))
    for j in range(1, R + 1):
        p.join(j)
    for j in range(1, R + 1):
        p.check_receiver_bytes(j)
    st = p.c.stats()
    assert st["kernel_launches"] == 1 and st["bytes_read_planned"] == nbytes and st["bytes_written_planned"] == R * nbytes
    p.close()


def test_more_receivers_than_one_wave_addresses():
    """1500 receivers of one object (a wave's table holds 1024 receiver addresses; the directory 4096 rows): the list is
    split over waves, every receiver gets the bytes, the source is read once per wave."""
    elems, R = 3 * 4096 + 5, 1500
    p = Pair(16 << 10, 2, 4, tau=3)
    p.create(0, 99, gen(("uniform",), 32, 0, elems))
    for j in range(1, R + 1):
        p.create(j, j % 50, nbytes=elems * 4, dtype=DT_F32)
    p.put(0)
    p.broadcast(0, list(range(1, R + 1)))
    for j in range(1, R + 1):
        p.join(j)
    p.check_schedule(0)
    for j in (1, 2, 1023, 1024, 1025, 1026, R - 1, R):
        p.check_receiver_bytes(j)
    src = p.dev[0].view(torch.uint8)
    for j in range(1, R + 1):
        assert torch.equal(p.dev[j], src), j
    st = p.c.stats()
    assert st["kernel_launches"] == 2 and st["bytes_written_planned"] == R * elems * 4
    p.close()


def test_a_small_object_is_spread_over_more_ctas_than_it_has_full_tiles():
    """256 KiB is 8 tiles of 32 KiB -- far fewer than there are CTAs: the wave uses 4 KiB tiles (64 of them); a 16 MiB
    object keeps the full tile.  Ragged sizes stay exact either way."""
    for nbytes, want_tiles in ((256 << 10, 64), ((256 << 10) + 36, 65), (16 << 20, 512)):
        p = Pair(1 << 20, 2, 2)
        p.create(0, 99, gen(("uniform",), 33, 0, nbytes // 4))
        for j in range(1, 5):
            p.create(j, j, nbytes=nbytes, dtype=DT_F32)
        p.put(0)
        p.broadcast(0, [1, 2, 3, 4])
        for j in range(1, 5):
            p.join(j)
        for j in range(1, 5):
            p.check_receiver_bytes(j)
        st = p.c.stats()
        assert st["kernel_launches"] == 1 and st["tiles"] == want_tiles, (nbytes, st["tiles"])
        p.close()


def test_partial_source_feeds_receivers_chunk_by_chunk():
    nbytes, chunk = 10 * 4096 + 40, 4096
    p = Pair(chunk, 2, 2)
    p.create(0, 99, gen(("uniform",), 2, 0, nbytes // 4))
    for j in range(1, 6):
        p.create(j, j, nbytes=nbytes, dtype=DT_F32)
    p.broadcast(0, [1, 2, 3, 4, 5])
    t = 0
    for step in range(1, 12):
        t += 50
        p.advance(t)
        p.put(0, min(nbytes, step * chunk))
        if step <= 5:
            p.join(step)
        p.progress()
    rc, _, _ = p.c.try_get(1)
    assert rc == hpl.HPL_OK
    for j in range(1, 6):
        p.check_receiver_bytes(j)
    p.check_schedule(0)
    p.close()


def test_receiver_failure_orphans_resume_and_bytes_match():
    nbytes, chunk, R = 64 * 4096, 4096, 8
    p = Pair(chunk, 2, 1, tau=100)
    p.create(0, 99, gen(("uniform",), 3, 0, nbytes // 4))
    for j in range(1, R + 1):
        p.create(j, j, nbytes=nbytes, dtype=DT_F32)
    p.put(0)
    p.broadcast(0, list(range(1, R + 1)))
    for j in range(1, 5):
        p.advance(j * 150)
        p.join(j)
    p.progress()
    p.advance(1500)
    p.fail(2)                       # receiver 2 was feeding receiver 3
    for j in range(5, R + 1):
        p.advance(1500 + j * 100)
        p.join(j)
    p.check_schedule(0)
    for j in range(1, R + 1):
        if j == 2:
            rc, _, _ = p.c.try_get(j)
            assert rc == hpl.HPL_ERR_FAILED_WORKER
        else:
            p.check_receiver_bytes(j)
    p.check_schedule(0)
    p.close()


def test_get_before_join_and_before_source_times_out():
    p = Pair(4096, 2, 2)
    p.create(0, 99, gen(("uniform",), 3, 0, 5000))
    p.create(1, 1, nbytes=20_000, dtype=DT_F32)
    p.create(2, 2, nbytes=20_000, dtype=DT_F32)
    p.broadcast(0, [1, 2])
    rc, _, _ = p.c.try_get(1)
    assert rc == hpl.HPL_ERR_TIMEOUT
    p.join(1)
    rc, _, _ = p.c.try_get(1)
    assert rc == hpl.HPL_ERR_TIMEOUT     # nothing has been put
    p.put(0)
    p.check_receiver_bytes(1)
    p.close()


def test_rebuilt_receiver_asks_again():
    nbytes, chunk = 32 * 4096, 4096
    p = Pair(chunk, 2, 1, tau=100)
    p.create(0, 99, gen(("uniform",), 8, 0, nbytes // 4))
    for j in range(1, 5):
        p.create(j, j, nbytes=nbytes, dtype=DT_F32)
    p.put(0)
    p.broadcast(0, [1, 2, 3, 4])
    for j in (1, 2, 3):
        p.advance(j * 120)
        p.join(j)
    p.progress()
    p.advance(1000)
    p.fail(2)
    p.advance(1500)
    p.c.rejoin(2)
    p.o.rejoin(2)
    # rebuilt, but it has not asked again: it holds no copy, although the copy it held before it failed was complete
    from oracle.store import StoreError, ERR_TIMEOUT
    with pytest.raises(StoreError) as ei:
        p.o.get(2)
    assert ei.value.code == ERR_TIMEOUT and p.c.try_get(2)[0] == hpl.HPL_ERR_TIMEOUT
    p.dev[2] = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    p.advance(1600)
    p.join(2)
    p.join(4)
    p.check_schedule(0)
    for j in (1, 2, 3, 4):
        p.check_receiver_bytes(j)
    p.check_schedule(0)
    p.close()


def _bcast_timeline(seed):
    """One broadcast under random events: a source that is put in instalments (from the device or from host memory), staggered
    joins, worker failures (the source's too), rebuilt workers that ask again or not, explicit progress, Gets in between."""
    rng = np.random.default_rng(seed)
    R, d, tau = int(rng.integers(1, 14)), int(rng.integers(1, 4)), int(rng.integers(1, 60))
    chunk = int(rng.choice([4096, 16384, 65536]))
    nbytes = int(rng.integers(1, 9)) * chunk + int(rng.choice([0, 0, 4, 1000, 4097]))
    nbytes -= nbytes % 4
    plan_ahead = bool(rng.random() < 0.3)
    p = Pair(chunk, 2, d, tau=tau, eager=bool(rng.random() < 0.4), plan_ahead=plan_ahead, poll_budget_ns=3_000_000 if plan_ahead else 0)
    nw = int(rng.integers(1, R + 2))
    host_src = rng.random() < 0.3
    data = gen(("uniform",), 900 + seed, 0, nbytes // 4)
    srcw = int(rng.integers(0, nw)) if rng.random() < 0.2 else 99
    if host_src:
        p.host[0] = data
        p.c.create(0, srcw, nbytes, DT_F32)
        p.o.create(0, srcw, nbytes, DT_F32)
    else:
        p.create(0, srcw, data)
    for j in range(1, R + 1):
        p.create(j, int(rng.integers(0, nw)), nbytes=nbytes, dtype=DT_F32)
    pref = 0

    def put(nb):
        if host_src:
            p.c.put_host(0, p.host[0].ctypes.data, nb)
            p.o.put(0, p.host[0], nb)
        else:
            p.put(0, nb)

    if rng.random() < 0.5:
        pref = nbytes if rng.random() < 0.6 else min(nbytes, int(rng.integers(0, nbytes // chunk + 1)) * chunk)
        if pref:
            put(pref)
    p.broadcast(0, list(range(1, R + 1)))
    joiners = list(rng.permutation(np.arange(1, R + 1)))
    t = 0

    def get(j):
        nonlocal t
        ro = OK
        try:
            want = p.o.get(j)
        except StoreError as e:
            ro = e.code
        rl, ptr, nb = p.c.try_get(j)
        if plan_ahead and ro == OK and rl == hpl.HPL_ERR_TIMEOUT:
            p.c.sync()
            rl, ptr, nb = p.c.try_get(j)
        assert rl == ro, (j, ro, rl)
        if ro == OK:
            assert p.view(ptr, nb).cpu().numpy().tobytes() == want.tobytes(), f"receiver {j} differs"
        t = max(t, p.o.now)
        if plan_ahead:
            p.c.sync()

    for s in range(int(rng.integers(R, 4 * R + 6))):
        t = max(t + int(rng.integers(0, 3 * tau)), p.o.now)
        p.advance(t)
        r = rng.random()
        if r < 0.4 and joiners:
            j = int(joiners.pop(0))
            if p.o.objects[j].alive:
                p.join(j)
        elif r < 0.55 and pref < nbytes and p.o.objects[0].alive:
            pref = nbytes if rng.random() < 0.5 else min(nbytes, pref + chunk)
            put(pref)
        elif r < 0.67:
            p.fail(int(rng.integers(0, nw)))
        elif r < 0.75:
            wk = int(rng.integers(0, nw))
            p.c.rejoin(wk)
            p.o.rejoin(wk)
            for j in range(1, R + 1):
                if p.o.objects[j].worker == wk and j not in joiners and rng.random() < 0.7:
                    joiners.append(j)
        elif r < 0.85:
            p.progress()
        else:
            get(int(rng.integers(1, R + 1)))
        p.check_schedule(0)
    if pref < nbytes and p.o.objects[0].alive:
        t = max(t + 1, p.o.now)
        p.advance(t)
        put(nbytes)
    for j in range(1, R + 1):
        get(j)
        p.check_schedule(0)
    if plan_ahead:
        p.c.sync()
    p.close()


@pytest.mark.parametrize("block", range(3))
def test_random_broadcast_timelines_match_the_oracle(block):
    for seed in range(block * 40, (block + 1) * 40):
        try:
            _bcast_timeline(seed)
        except AssertionError as e:
            raise AssertionError(f"seed {seed}: {e}") from e


def test_receivers_keep_what_the_schedule_gave_them_when_the_source_is_lost_before_any_copy_ran():
    """Copies are made lazily; in the schedule the receivers had the whole object when the source's worker failed.  The
    failure itself enqueues the copies that copy can still serve."""
    nbytes, chunk = 5 * 4096 + 8, 4096
    p = Pair(chunk, 2, 2, tau=10)
    p.create(0, 7, gen(("uniform",), 12, 0, nbytes // 4))
    for j in (1, 2, 3):
        p.create(j, 10 + j, nbytes=nbytes, dtype=DT_F32)
    p.put(0)
    p.broadcast(0, [1, 2, 3])
    for j in (1, 2, 3):
        p.join(j)
    p.advance(100_000)                                  # every transfer of the schedule has landed; nothing has run yet
    assert p.c.stats()["kernel_launches"] == 0
    p.fail(7)
    for j in (1, 2, 3):
        p.check_receiver_bytes(j)
    p.check_schedule(0)
    p.close()
