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


@pytest.mark.parametrize("fuse_fanout", [True, False])
def test_allreduce_is_reduce_then_broadcast(fuse_fanout):
    elems, chunk, R = 5 * 4096 + 12, 16 << 10, 6
    p = Pair(chunk, 2, 2, tau=50, fuse_fanout=fuse_fanout)
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


@pytest.mark.parametrize("dtype,k,R,elems,chunk,d", [("f32", 8, 8, 3 * 4096 + 7, 16 << 10, 2), ("bf16", 8, 8, 70_001, 32 << 10, 2),
                                                     ("bf16", 64, 64, 24_576, 16 << 10, 4), ("f32", 3, 5, 6, 4096, 1),
                                                     ("f32", 1, 3, 5000, 4096, 2), ("bf16", 5, 130, 9000, 8 << 10, 4)])
def test_fused_allreduce_every_receiver_holds_the_target_bits(dtype, k, R, elems, chunk, d):
    """Reduce followed by broadcast with all receivers joined before anything runs: one pass writes the target and every
    receiver (ragged tiles, bf16 inputs whose chunks are twice the output's, more receivers than one wave serves)."""
    p = Pair(chunk, d, 2)
    code = DT_BF16 if dtype == "bf16" else DT_F32
    for i in range(k):
        p.create(i, i, gen(("uniform",) if dtype == "f32" else ("normal", 0.02), 97, i, elems, dtype))
    for j in range(R):
        p.create(1000 + j, 500 + j, nbytes=elems * 4, dtype=DT_F32)
    p.reduce(100, list(range(k)), k, 0, code)
    p.broadcast(100, [1000 + j for j in range(R)])
    for j in range(R):
        p.join(1000 + j)
    p.advance(5)
    for i in range(k):
        p.put(i)
    want = p.check_target_bits(100).cpu().numpy()
    for j in range(R):
        p.check_receiver_bytes(1000 + j)
        assert p.dev[1000 + j].view(torch.uint8).cpu().numpy().tobytes() == want.tobytes()
    st = p.c.stats()
    assert st["fused_fanout_tasks"] >= 1 and st["bytes_read_planned"] <= k * p.host[0].nbytes + max(0, R - 128) * elems * 4
    assert st["bytes_written_planned"] == (R + 1) * elems * 4
    p.close()


def test_fused_allreduce_with_a_member_lost_half_way_is_redone_for_target_and_receivers():
    elems, chunk, k, R = 8 * 4096 + 5, 16 << 10, 6, 4
    p = Pair(chunk, 2, 2)
    for i in range(k + 1):
        p.create(i, i, gen(("uniform",), 98, i, elems))
    for j in range(R):
        p.create(1000 + j, 500 + j, nbytes=elems * 4, dtype=DT_F32)
    p.reduce(100, list(range(k + 1)), k)               # object k is the spare
    p.broadcast(100, [1000 + j for j in range(R)])
    for j in range(R):
        p.join(1000 + j)
    for i in range(k):
        p.advance(i + 1)
        p.put(i, 4 * chunk)                            # half of every object
    p.progress()                                       # half of the result is in the target and in the receivers
    assert p.c.stats()["fused_fanout_tasks"] >= 1
    p.advance(50)
    p.fail(2)
    p.advance(60)
    p.put(k)
    for i in range(k):
        if i != 2:
            p.put(i)
    want = p.check_target_bits(100).cpu().numpy()
    p.check_schedule(100)
    for j in range(R):
        p.check_receiver_bytes(1000 + j)
        assert p.dev[1000 + j].view(torch.uint8).cpu().numpy().tobytes() == want.tobytes()
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
