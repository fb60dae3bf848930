"""Chunks consumed while they are still arriving: host objects copied into the store chunk by chunk,
kernels that poll the directory's progress counters, and the bound on every such wait."""
import numpy as np
import pytest
import torch

import paper_2002_05814_b200 as hpl
from oracle import values as ov
from oracle.store import DT_F32, DT_BF16
from tests.harness import Pair, gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2002_05814_b200 import build
    build.build()
    assert torch.cuda.is_available()


def _pinned(a: np.ndarray) -> torch.Tensor:
    t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
    return t.pin_memory()


@pytest.mark.parametrize("plan_ahead", [True, False])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_host_objects_are_copied_in_reduced_and_read_back(plan_ahead, dtype):
    k, elems, chunk = 8, 300_003 if dtype == "f32" else 300_008, 64 << 10
    p = Pair(chunk, 2, plan_ahead=plan_ahead, arena_bytes=128 << 20)
    code = DT_BF16 if dtype == "bf16" else DT_F32
    host = {}
    for i in range(k):
        a = gen(("normal", 0.02), 70, i, elems, dtype)
        p.host[i] = a
        host[i] = _pinned(a)
        p.c.create(i, i, a.nbytes, code)
        p.o.create(i, i, a.nbytes, code)
    p.c.reduce(100, list(range(k)), k, 0, code)
    p.o.reduce(100, list(range(k)), k, 0, code)
    for i in range(k):
        half = (a.nbytes // 2) // chunk * chunk
        p.c.put_host(i, host[i].data_ptr(), half)          # the copy is published in two instalments
        p.o.put(i, p.host[i], half)
    if plan_ahead:
        p.c.progress()                                       # the kernel starts before the objects are complete
    for i in range(k):
        p.c.put_host(i, host[i].data_ptr(), p.host[i].nbytes)
        p.o.put(i, p.host[i], p.host[i].nbytes)
    out = torch.empty(elems, dtype=torch.float32).pin_memory()
    p.c.get_host(100, out.data_ptr(), elems * 4)
    want = p.o.get(100)
    assert np.array_equal(out.numpy().view(np.uint32), want.view(np.uint32))
    st = p.c.stats()
    assert st["h2d_bytes"] == k * p.host[0].nbytes and st["d2h_bytes"] == elems * 4 and st["device_timeouts"] == 0
    p.check_schedule(100)
    p.close()


def test_host_source_is_broadcast_while_it_is_copied_in():
    nbytes, R = 3 << 20, 6
    p = Pair(256 << 10, 2, 2, plan_ahead=True, arena_bytes=64 << 20)
    a = gen(("uniform",), 71, 0, nbytes // 4)
    p.host[0] = a
    pin = _pinned(a)
    p.c.create(0, 99, nbytes, DT_F32)
    p.o.create(0, 99, nbytes, DT_F32)
    for j in range(1, R + 1):
        p.create(j, j, nbytes=nbytes, dtype=DT_F32)
    p.broadcast(0, list(range(1, R + 1)))
    p.c.put_host(0, pin.data_ptr(), 1 << 20)
    p.o.put(0, a, 1 << 20)
    for j in range(1, R + 1):
        p.join(j)
    p.c.progress()
    p.c.put_host(0, pin.data_ptr(), nbytes)
    p.o.put(0, a, nbytes)
    for j in range(1, R + 1):
        p.check_receiver_bytes(j)
    assert p.c.stats()["device_timeouts"] == 0
    p.close()


def test_polling_kernel_picks_up_chunks_published_while_it_runs():
    k, elems, chunk = 4, 16 * 4096, 16 << 10                 # 16 chunks of 4096 elements
    p = Pair(chunk, 2, plan_ahead=True, poll_budget_ns=500_000_000)
    for i in range(k):
        p.create(i, i, gen(("uniform",), 72, i, elems))
    p.reduce(100, list(range(k)), k)
    for i in range(k):
        p.put(i, 4 * chunk)                                  # a quarter of every object
    p.progress()                                             # planned for all 16 chunks: the kernel now waits at chunk 4
    for step in (8, 12, 16):
        for i in range(k):
            p.put(i, step * chunk)                           # counters travel on the control stream
    p.check_target_bits(100)
    st = p.c.stats()
    assert st["device_timeouts"] == 0 and st["kernel_launches"] == 1
    p.close()


def test_a_wait_nothing_ends_runs_out_and_the_context_stays_usable():
    k, elems, chunk = 3, 10 * 4096, 16 << 10
    p = Pair(chunk, 2, plan_ahead=True, poll_budget_ns=3_000_000)    # 3 ms
    for i in range(k):
        p.create(i, i, gen(("uniform",), 73, i, elems))
    p.reduce(100, list(range(k)), k)
    p.put(0)
    p.put(1)
    p.put(2, 2 * chunk)                                      # object 2 stops at chunk 2 and nothing advances it
    rc, _, _ = p.c.try_get(100)
    assert rc == hpl.HPL_ERR_TIMEOUT                          # the host already knows the target cannot complete
    assert p.c.sync() == hpl.HPL_ERR_TIMEOUT                  # ... and the kernel's bounded wait has run out
    assert p.c.stats()["device_timeouts"] == 1
    x = torch.ones(1024, device="cuda")                       # the device is fine
    assert float(x.sum()) == 1024.0
    p.put(2)                                                  # the rest arrives: everything is planned again
    p.check_target_bits(100)
    assert p.c.sync() == hpl.HPL_OK
    p.close()


def test_eager_mode_runs_what_became_runnable_at_every_event():
    k, elems = 8, 30_000
    p = Pair(32 << 10, 2, 2, eager=True)
    for i in range(k):
        p.create(i, i, gen(("uniform",), 74, i, elems))
    for j in range(3):
        p.create(50 + j, 20 + j, nbytes=elems * 4, dtype=DT_F32)
    p.reduce(100, list(range(k)), k)
    p.broadcast(100, [50, 51, 52])
    p.join(50)
    launches = []
    for t, i in enumerate([2, 5, 0, 7, 1, 3, 6, 4]):
        p.advance(t + 1)
        p.put(i)                                   # no explicit hpl_progress anywhere
        launches.append(p.c.stats()["kernel_launches"])
    assert launches[0] == 0 and launches[1] >= 1 and launches[-1] > launches[1]   # subtrees are reduced as they complete
    p.join(51)
    p.join(52)
    p.check_target_bits(100)
    for j in range(3):
        p.check_receiver_bytes(50 + j)
    p.close()


def test_delete_returns_memory_and_rows_for_the_next_round():
    p = Pair(16 << 10, 2, 2, arena_bytes=8 << 20)       # room for one round only: every round must give it back
    base = p.c.stats()["arena_used"]
    for rnd in range(6):
        ids = [10 * rnd + i for i in range(4)]
        for i in ids:
            p.create(i, i % 4, gen(("uniform",), 75 + rnd, i, 300_000))
        p.reduce(1000 + rnd, ids, 4)
        for i in ids:
            p.put(i)
            p.progress()
        p.check_target_bits(1000 + rnd)
        assert p.c.stats()["arena_used"] > base
        for i in [1000 + rnd] + ids:
            p.c.delete(i)
            p.o.delete(i)
        assert p.c.stats()["arena_used"] == base
    p.close()


def test_waits_are_counted():
    p = Pair(16 << 10, 2, plan_ahead=True, poll_budget_ns=500_000_000)
    for i in range(2):
        p.create(i, i, gen(("uniform",), 76, i, 8 * 4096))
    p.reduce(100, [0, 1], 2)
    p.put(0)
    p.put(1, 16 << 10)
    p.progress()
    import time
    time.sleep(0.05)                                # the kernel is polling for chunk 1 of object 1
    p.put(1)
    p.check_target_bits(100)
    assert p.c.stats()["device_waits"] >= 1 and p.c.stats()["device_timeouts"] == 0
    p.close()


def test_pageable_host_memory_and_get_host_of_every_kind_of_object():
    elems, chunk = 50_000, 32 << 10
    p = Pair(chunk, 2, 2, arena_bytes=32 << 20)
    a = [gen(("uniform",), 77, i, elems) for i in range(3)]        # ordinary (pageable) numpy memory
    for i in range(3):
        p.host[i] = a[i]
        p.c.create(i, i, a[i].nbytes, DT_F32)
        p.o.create(i, i, a[i].nbytes, DT_F32)
        p.c.put_host(i, a[i].ctypes.data, a[i].nbytes)
        p.o.put(i, a[i], a[i].nbytes)
    p.create(9, 9, nbytes=elems * 4, dtype=DT_F32)
    p.reduce(100, [0, 1, 2], 3)
    p.broadcast(1, [9])
    p.join(9)
    out = np.empty(elems, np.float32)
    p.c.get_host(100, out.ctypes.data, out.nbytes)                   # a Reduce output
    assert np.array_equal(out.view(np.uint32), p.o.get(100).view(np.uint32))
    p.c.get_host(9, out.ctypes.data, out.nbytes)                     # a broadcast copy
    assert out.tobytes() == a[1].tobytes()
    p.c.get_host(2, out.ctypes.data, out.nbytes)                     # a put object (its copy in the store)
    assert out.tobytes() == a[2].tobytes()
    with pytest.raises(hpl.HplError) as ei:
        p.c.get_host(2, out.ctypes.data, 16)                         # destination too small
    assert ei.value.code == hpl.HPL_ERR_INVALID
    p.close()


def test_many_device_puts_then_a_host_object_with_plan_ahead():
    """The control stream is busy with the rows of many device objects when a host object is put: its row must reach
    the directory with a zero counter (a snapshot taken at the Put), so that the polling wave never sees chunks that
    have not landed."""
    elems, chunk, k = 24 * 4096 + 9, 16 << 10, 41
    for rnd in range(3):
        p = Pair(chunk, 4, plan_ahead=True, poll_budget_ns=500_000_000, arena_bytes=64 << 20)
        for i in range(k):
            p.create(i, i, gen(("uniform",), 78 + rnd, i, elems))
        p.reduce(100, list(range(k)), k)
        for i in range(k - 1):
            p.put(i)                                         # device objects: rows and counters on the control stream
        host = torch.from_numpy(p.host[k - 1]).pin_memory()
        p.c.put_host(k - 1, host.data_ptr(), host.numel() * 4)   # copied in chunk by chunk behind them
        p.o.put(k - 1, p.host[k - 1], p.host[k - 1].nbytes)
        p.progress()
        p.check_target_bits(100)
        assert p.c.stats()["device_timeouts"] == 0
        p.close()


def test_plan_ahead_put_publishes_what_is_visible_at_the_call():
    """The documented contract of hpl_put with plan_ahead = 1: the prefix must be valid when the call is made.  A
    producer that fills the object on another stream synchronises before each Put; the polling wave, launched before
    any byte existed, then consumes each piece as its counter arrives."""
    elems, chunk = 32 * 4096, 16 << 10
    p = Pair(chunk, 2, plan_ahead=True, poll_budget_ns=500_000_000)
    src = gen(("uniform",), 79, 0, elems)
    other = gen(("uniform",), 79, 1, elems)
    p.create(1, 1, other)
    p.put(1)
    p.host[0] = src
    buf = torch.zeros(elems, dtype=torch.float32, device="cuda")
    p.dev[0] = buf
    p.c.create(0, 0, elems * 4, DT_F32)
    p.o.create(0, 0, elems * 4, DT_F32)
    p.reduce(100, [0, 1], 2)
    whole = torch.from_numpy(src).cuda()
    side = torch.cuda.Stream()
    p.c.put(0, buf.data_ptr(), 0)                            # published with nothing valid yet: the arrival
    p.o.put(0, src, 0)
    p.progress()                                             # the wave polls for chunk 0 of object 0
    for step in (8, 20, 32):
        with torch.cuda.stream(side):
            buf[: step * 4096].copy_(whole[: step * 4096])
        side.synchronize()                                   # visible at the call
        p.c.put(0, buf.data_ptr(), step * chunk)
        p.o.put(0, src, step * chunk)
    p.check_target_bits(100)
    assert p.c.stats()["device_timeouts"] == 0
    p.close()


def test_arena_canaries_notice_a_write_behind_a_block():
    """The overrun detector of the test harness itself: the test (not a kernel) changes one byte behind a reduce target
    inside the arena it owns; hpl_check_guards reports it."""
    p = Pair(16 << 10, 2)
    for i in range(2):
        p.create(i, i, gen(("uniform",), 80, i, 1000))
        p.put(i)
    p.reduce(100, [0, 1], 2)
    ptr, n = p.c.get(100)
    assert p.c.check_guards() == 0
    off = ptr - p.arena.data_ptr()
    p.arena[off + n + 3] = 0x11
    torch.cuda.synchronize()
    assert p.c.check_guards() == 1
    p.c.shutdown()


def test_partial_results_are_evicted_least_recently_used_when_the_arena_is_full():
    """Section 6: pinned copies (sources, outputs) stay, other copies go under memory pressure.  Two Reduces whose tree
    nodes each keep their reduced object do not fit the arena together: the second one's buffers take the place of the
    first one's partial results, and after a failure the first one makes its own again."""
    elems, chunk, k = 64 * 1024, 64 << 10, 8
    S = elems * 4
    fixed = 4096 * 32 + 256 * 32 + (64 << 10)              # directory, error records, slack
    p = Pair(chunk, 2, fuse=False, arena_bytes=fixed + 7 * (S + 512))   # room for 7 buffers; the two trees want 2 x 4
    for i in range(2 * k + 1):
        p.create(i, i, gen(("uniform",), 81, i, elems))
        p.put(i)
    p.reduce(100, list(range(k)) + [2 * k], k)              # object 16 is a spare
    p.check_target_bits(100)
    assert p.c.stats()["evictions"] == 0
    p.reduce(200, list(range(k, 2 * k)), k)
    p.check_target_bits(200)
    ev = p.c.stats()["evictions"]
    assert ev >= 1
    p.advance(10)
    p.fail(3)                                               # the first tree has to redo the path above object 3
    p.check_target_bits(100)
    p.check_schedule(100)
    assert p.c.stats()["evictions"] > ev
    p.check_target_bits(200)                                # outputs were never touched
    p.close()


def test_a_pass_that_runs_out_of_arena_leaves_nothing_noted_as_done():
    """The arena holds two outputs and nothing else.  A Get of the Reduce finds its first chunk computable in one fused
    pass and, for the chunks behind it, needs a buffer for an inner node -- which the arena cannot give: the Get says so,
    and nothing of that pass counts as done.  Once the other output is deleted the same Get computes every chunk."""
    elems, chunk = 64 * 1024, 64 << 10                      # four chunks; an object is larger than the arena's slack
    S = elems * 4
    fixed = 4096 * 32 + 256 * 32 + (64 << 10)              # directory, error records, slack
    p = Pair(chunk, 2, fuse=True, arena_bytes=fixed + 2 * (S + 512))
    for i in range(6):
        p.create(i, i, gen(("uniform",), 83, i, elems))
    p.put(4)
    p.put(5)
    p.reduce(900, [4, 5], 2)                                # its output fills the second half of the arena
    p.check_target_bits(900)
    p.reduce(100, [0, 1, 2, 3], 4)
    p.advance(1)
    p.put(0)                                                # first arrival: position 3, the leaf under position 1
    p.advance(2)
    p.put(1)                                                # position 1: that node has everything it needs
    p.advance(3)
    p.put(2, chunk)                                         # the root's own object, first chunk only
    p.advance(4)
    p.put(3, chunk)                                         # position 2, first chunk only
    assert p.o.reduces[100]["sched"].obj_at == [2, 1, 3, 0]
    assert p.c.try_get(100)[0] == hpl.HPL_ERR_NOMEM
    assert p.c.try_get(100)[0] == hpl.HPL_ERR_NOMEM         # and again: the state is as before the attempt
    p.delete(900)
    p.advance(5)
    p.put(2)
    p.put(3)
    p.check_target_bits(100)
    p.check_schedule(100)
    p.close()


def test_a_wait_that_runs_out_voids_its_own_collective_and_its_consumers_only():
    """plan_ahead: Reduce A waits for chunks of an object that never come; Reduce C consumes A's output; Reduce B, requested
    after both, has nothing to do with them.  Every Get plans A again and A's wave gives up again -- B's result, computed
    once, stands and is returned; C cannot complete; when the object finally arrives everything completes."""
    elems, chunk = 6 * 4096, 16 << 10
    p = Pair(chunk, 2, plan_ahead=True, poll_budget_ns=2_000_000)
    for i in range(6):
        p.create(i, i, gen(("uniform",), 82, i, elems))
    p.reduce(100, [0, 1], 2)                       # A
    p.reduce(300, [100, 2], 2)                     # C consumes A
    p.reduce(200, [3, 4, 5], 3)                    # B, independent
    p.put(0)
    p.put(1, chunk)                                # published, one chunk of six valid: A's wave will wait for the rest
    for i in (2, 3, 4, 5):
        p.put(i)
    p.check_target_bits(200)                       # B completes although A's wave runs out in the same pass
    launches = p.c.stats()["kernel_launches"]
    for _ in range(3):
        assert p.c.try_get(100)[0] == hpl.HPL_ERR_TIMEOUT and p.c.try_get(300)[0] == hpl.HPL_ERR_TIMEOUT
        p.check_target_bits(200)                   # ... and is not computed again
    st = p.c.stats()
    assert st["device_timeouts"] >= 3
    p.put(1)
    p.check_target_bits(100)
    p.check_target_bits(300)
    p.check_target_bits(200)
    p.close()
