"""Composed collectives on the GPU: a Reduce whose input is another Reduce's output, and reduce
followed by broadcast (allreduce), streamed chunk by chunk through the directory."""
import numpy as np
import pytest
import torch

import paper_2002_05814_b200 as hpl
from oracle.store import DT_F32, DT_BF16
from tests.harness import Pair, gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2002_05814_b200 import build
    build.build()
    assert torch.cuda.is_available()


@pytest.mark.parametrize("fuse", [True, False])
def test_reduce_of_a_reduce_output_streams_through(fuse):
    elems, chunk = 6 * 4096 + 77, 16 << 10           # 7 chunks, the last one short
    p = Pair(chunk, 2, fuse=fuse)
    for i in range(7):
        p.create(i, i, gen(("uniform",), 90, i, elems))
    p.reduce(100, [0, 1, 2, 3], 3)                    # three of four
    p.reduce(200, [100, 4, 5, 6], 4)                  # its output is an input here
    nbytes = elems * 4
    t = 0
    for step in (2, 4, 7):                            # prefixes grow: the first output is consumed while partial
        for i in (0, 2, 3, 4, 5, 6):
            t += 3
            p.advance(t)
            p.put(i, min(nbytes, step * chunk))
        p.progress()
    p.check_schedule(100)
    p.check_schedule(200)
    p.check_target_bits(100)
    p.check_target_bits(200)
    assert p.c.stats()["kernel_launches"] >= 4
    p.close()


def test_bf16_first_stage_feeds_an_fp32_second_stage():
    elems = 3 * 4096 + 8
    p = Pair(8 << 10, 4)
    for i in range(5):
        p.create(i, i, gen(("normal", 0.02), 91, i, elems, "bf16"))
        p.put(i)
    extra = gen(("uniform",), 92, 9, elems)
    p.create(9, 9, extra)
    p.put(9)
    p.reduce(100, [0, 1, 2, 3, 4], 5, 0, DT_BF16)
    p.reduce(200, [100, 9], 2, 0, DT_F32)
    p.check_target_bits(200)
    p.close()


def test_allreduce_is_reduce_then_broadcast():
    elems, chunk, R = 5 * 4096 + 12, 16 << 10, 6
    p = Pair(chunk, 2, 2, tau=50)
    for i in range(4):
        p.create(i, i, gen(("uniform",), 93, i, elems))
    for j in range(R):
        p.create(50 + j, 20 + j, nbytes=elems * 4, dtype=DT_F32)
    p.reduce(100, [0, 1, 2, 3], 4)
    p.broadcast(100, [50 + j for j in range(R)])
    p.join(50)
    p.join(51)
    nbytes = elems * 4
    t = 0
    for step in (1, 3, 6):
        for i in range(4):
            t += 10
            p.advance(t)
            p.put(i, min(nbytes, step * chunk))
        p.progress()                                   # reduced chunks flow on to the receivers that have joined
        if step == 3:
            p.join(52)
    for j in range(3, R):
        t += 500
        p.advance(t)
        p.join(50 + j)
    p.check_schedule(100)
    want = p.check_target_bits(100).cpu().numpy()
    for j in range(R):
        p.check_receiver_bytes(50 + j)
        assert p.dev[50 + j].view(torch.uint8).cpu().numpy().tobytes() == want.tobytes()
    p.check_schedule(100)
    p.close()


def test_upstream_failure_voids_what_was_derived_from_the_output():
    elems = 20_000
    p = Pair(16 << 10, 2, 2)
    for i in range(6):
        p.create(i, i, gen(("smallint", 100), 94, i, elems))
    p.create(60, 30, nbytes=elems * 4, dtype=DT_F32)
    p.reduce(100, [0, 1, 2, 5], 3)
    p.reduce(200, [100, 3, 4], 3)
    p.broadcast(200, [60])
    for i in (0, 1, 2, 3, 4):
        p.put(i)
    p.join(60)
    p.check_target_bits(200)
    p.check_receiver_bytes(60)
    p.advance(p.o.now + 100)                           # the Get let virtual time run
    p.fail(1)                                          # a member of the first Reduce; object 5 is the spare
    rc, _, _ = p.c.try_get(60)
    assert rc == hpl.HPL_ERR_TIMEOUT
    p.put(5)
    got = p.check_target_bits(200).cpu().numpy()
    assert np.array_equal(got, sum(p.host[i] for i in (0, 5, 2, 3, 4)))
    p.check_receiver_bytes(60)
    assert p.dev[60].view(torch.float32).cpu().numpy().tobytes() == got.tobytes()
    p.close()
