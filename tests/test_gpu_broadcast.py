"""Parity of the CUDA broadcast path with the oracle (through the C ABI), byte by byte."""
import numpy as np
import pytest
import torch

import paper_2002_05814_b200 as hpl
import workloads as wl
from oracle.store import DT_F32, DT_BF16
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
    p.dev[2] = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    p.advance(1600)
    p.join(2)
    p.join(4)
    p.check_schedule(0)
    for j in (1, 2, 3, 4):
        p.check_receiver_bytes(j)
    p.check_schedule(0)
    p.close()
