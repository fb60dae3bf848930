"""The planners (host logic) on a machine without a GPU.  A context created without an arena plans exactly
as it would with one -- its tasks are counted in the statistics -- but launches nothing."""
import math

import pytest

import paper_2002_05814_b200 as hpl
import workloads as wl
from paper_2002_05814_b200 import build as hpl_build


@pytest.fixture(scope="module", autouse=True)
def _built():
    hpl_build.build()


def _addr(i):
    return 1 << 20 | (i + 1) << 24          # distinct, 16-byte aligned, never dereferenced


def _plan_get(c, oid):
    rc, _, _ = c.try_get(oid)
    assert rc == hpl.HPL_ERR_CUDA            # planned to completion; only the device is missing
    return c.stats()


@pytest.mark.parametrize("name", ["cfg1", "cfg3", "cfg4"])
def test_everything_ready_is_one_fused_pass_with_exactly_the_algorithmic_bytes(name):
    w = wl.workload(name)
    dt = hpl.HPL_BF16 if w.dtype == "bf16" else hpl.HPL_F32
    with hpl.Context(w.chunk_bytes, w.degree, w.degree) as c:
        S = w.object_bytes
        for i in range(w.n_objects):
            c.create(i, i, S, dt)
        c.reduce(900, list(range(w.n_objects)), w.k, hpl.HPL_SUM, dt)
        for i in range(w.n_objects):
            c.advance(i)
            c.put(i, _addr(i), S)
        st = _plan_get(c, 900)
        assert st["reduce_tasks"] == 1 and st["kernel_launches"] == 1
        assert st["bytes_read_planned"] == w.k * S and st["bytes_written_planned"] == w.elems * 4


def test_broadcast_to_all_joined_receivers_reads_the_source_once():
    w = wl.workload("cfg4")
    S = w.object_bytes
    with hpl.Context(w.chunk_bytes, w.degree, w.degree) as c:
        c.create(0, 99, S, hpl.HPL_BF16)
        c.put(0, _addr(0), S)
        ids = list(range(1, 65))
        c.create_batch(ids, ids, S, hpl.HPL_BF16)
        c.broadcast(0, ids)
        c.join_batch(ids, [_addr(i) for i in ids])
        st = _plan_get(c, 64)
        assert st["fanout_tasks"] == 1 and st["bytes_read_planned"] == S and st["bytes_written_planned"] == 64 * S
        # a receiver that joins later is served from its sender's copy, not from the source again
        c.create(70, 70, S, hpl.HPL_BF16)


@pytest.mark.parametrize("d", [2, 4])
def test_progress_after_every_arrival_leaves_little_for_the_last_pass(d):
    k, S = 16, 1 << 20
    with hpl.Context(64 << 10, d, 2) as c:
        for i in range(k):
            c.create(i, i, S)
        c.reduce(900, list(range(k)), k)
        reads = []
        for i in range(k):
            c.advance(i + 1)
            c.put(i, _addr(i), S)
            c.progress()
            reads.append(c.stats()["bytes_read_planned"])
        st = _plan_get(c, 900)
        assert reads[-1] - reads[-2] <= (math.ceil(math.log(k, d)) + d) * S     # only the root path was left
        assert st["bytes_read_planned"] < 3 * k * S                             # merging early costs re-reads, boundedly


def test_failure_without_fusion_recomputes_only_the_root_paths():
    k, S, chunk = 32, 1 << 20, 64 << 10
    with hpl.Context(chunk, 2, 2, fuse=False) as c:
        for i in range(k):
            c.create(i, i, S)
        c.reduce(900, list(range(k)), k)
        for i in range(k):
            c.put(i, _addr(i), S if i != 7 else 6 * chunk)
        c.progress()
        before = c.stats()
        c.advance(5)
        c.fail(7)
        st = _plan_get(c, 900)
        redone = st["reduce_tasks"] - before["reduce_tasks"]
        assert redone <= 2 * 2 * (math.ceil(math.log2(k)) + 1)
        assert st["bytes_read_planned"] - before["bytes_read_planned"] < (k - 1) * S


def test_a_tree_larger_than_one_task_is_cut_and_launched_in_levels():
    k, S = 1000, 8192
    with hpl.Context(4096, 2, 2) as c:
        for i in range(k):
            c.create(i, i % 5, S)
            c.put(i, _addr(i), S)
        c.reduce(5000, list(range(k)), k)
        st = _plan_get(c, 5000)
        assert st["reduce_tasks"] > 1 and st["kernel_launches"] >= 2
        assert st["bytes_read_planned"] >= k * S
    with hpl.Context(4096, 1000, 2) as c:
        for i in range(800):
            c.create(i, 0, 64)
        with pytest.raises(hpl.HplError) as ei:
            c.reduce(5000, list(range(800)), 800)
        assert ei.value.code == hpl.HPL_ERR_INVALID


@pytest.mark.parametrize("fuse_fanout", [False, True])
def test_composed_collectives_are_planned_in_creation_order(fuse_fanout):
    S = 1 << 18
    with hpl.Context(64 << 10, 2, 2, fuse_fanout=fuse_fanout) as c:
        for i in range(6):
            c.create(i, i, S)
            c.put(i, _addr(i), S)
        c.reduce(100, [0, 1, 2], 3)
        c.reduce(200, [100, 3, 4, 5], 4)
        c.create(300, 50, S)
        c.broadcast(200, [300])
        c.join(300, _addr(30))
        st = _plan_get(c, 300)
        if fuse_fanout:      # the second stage's result goes to its target and to the receiver in the same pass
            assert st["reduce_tasks"] == 2 and st["fanout_tasks"] == 0 and st["fused_fanout_tasks"] == 1
            assert st["bytes_read_planned"] == 3 * S + 4 * S and st["bytes_written_planned"] == 3 * S
            assert st["kernel_launches"] == 2
        else:
            assert st["reduce_tasks"] == 2 and st["fanout_tasks"] == 1
            assert st["bytes_read_planned"] == 3 * S + 4 * S + S      # inputs of each stage, then the output once


def test_allreduce_of_8_to_8_is_one_pass_that_never_reads_the_target():
    """Reduce followed by broadcast (Section 3.4.3) with every receiver joined: k objects read, the result written to
    the target and to each receiver, one launch."""
    S, k, R = 1 << 20, 8, 8
    with hpl.Context(64 << 10, 2, 2) as c:
        for i in range(k):
            c.create(i, i, S)
            c.put(i, _addr(i), S)
        c.reduce(100, list(range(k)), k)
        for j in range(R):
            c.create(200 + j, 50 + j, S)
        c.broadcast(100, [200 + j for j in range(R)])
        for j in range(R):
            c.join(200 + j, _addr(40 + j))
        st = _plan_get(c, 200)
        assert st["kernel_launches"] == 1 and st["reduce_launches"] == 1 and st["fanout_launches"] == 0
        assert st["bytes_read_planned"] == k * S and st["bytes_written_planned"] == (R + 1) * S


def test_small_collectives_planned_in_one_pass_share_their_launches():
    """Objects under 64 KiB (Section 3.2's small objects): 32 Reduces and 8 broadcasts requested together are served by
    a few shared waves instead of one launch each; a Reduce that consumes another's output sits one stage later."""
    S = 4096
    with hpl.Context(64 << 10, 2, 2) as c:
        oid = 0
        for r in range(32):
            ids = list(range(oid, oid + 4))
            oid += 4
            for i in ids:
                c.create(i, i, S)
                c.put(i, _addr(i), S)
            c.reduce(10_000 + r, ids, 4)
        c.reduce(20_000, [10_000, 10_001], 2)              # composed: one stage behind its producers
        for b in range(8):
            c.create(30_000 + b, 900, S)
            c.put(30_000 + b, _addr(7), S)
            c.create(31_000 + b, 901 + b, S)
            c.broadcast(30_000 + b, [31_000 + b])
            c.join(31_000 + b, _addr(9))
        c.progress()
        st = c.stats()
        assert st["reduce_tasks"] == 33 and st["fanout_tasks"] == 8
        assert st["reduce_launches"] == 3 and st["fanout_launches"] == 1     # 24 + 8 tasks, then the composed one; 8 fan-outs
    with hpl.Context(64 << 10, 2, 2) as c:                 # objects above the threshold keep launches of their own
        for r in range(3):
            ids = list(range(4 * r, 4 * r + 4))
            for i in ids:
                c.create(i, i, 128 << 10)
                c.put(i, _addr(i), 128 << 10)
            c.reduce(10_000 + r, ids, 4)
        c.progress()
        assert c.stats()["reduce_launches"] == 3


def test_directory_rows_run_out_gracefully_and_come_back_with_delete():
    """The device directory has 4096 rows, one per published object.  The Put that finds none free says so and changes
    nothing; after a Delete the same Put goes through; a wider star than a task holds is refused at the request."""
    c = hpl.Context(4096, 2, 2)
    n = 4096 + 3
    for i in range(n):
        c.create(i, i, 4096)
    for i in range(4096):
        c.put(i, 4096 * (i + 1), 4096)
    with pytest.raises(hpl.HplError) as e:
        c.put(4096, 4096 * 5000, 4096)
    assert e.value.code == hpl.HPL_ERR_NOMEM
    with pytest.raises(hpl.HplError) as e:
        c.reduce(9000, [0, 1], 2)                      # the output needs a row as well
    assert e.value.code == hpl.HPL_ERR_NOMEM
    c.delete(7)
    c.put(4096, 4096 * 5000, 4096)
    c.delete(8)
    c.reduce(9000, [0, 1], 2)
    c.progress()
    assert c.stats()["reduce_tasks"] == 1
    c.shutdown()
    c = hpl.Context(4096, 1000, 2)
    for i in range(700):
        c.create(i, i, 4096)
    with pytest.raises(hpl.HplError) as e:
        c.reduce(9000, list(range(700)), 700)          # 699 children of one node
    assert e.value.code == hpl.HPL_ERR_INVALID
    c.reduce(9001, list(range(600)), 600)              # 599 children fit
    c.shutdown()
