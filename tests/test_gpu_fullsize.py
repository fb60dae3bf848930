"""The configurations at full size, in the launch configuration the benchmark times, checked on
sampled windows the oracle computes one by one (inputs are regenerated per window from the seeded
recipe), plus whole-buffer properties that hold at any size."""
import math

import numpy as np
import pytest
import torch

import paper_2002_05814_b200 as hpl
import workloads as wl
from oracle import reduce_tree as ort
from oracle import values as ov
from oracle.store import OracleStore, DT_F32, DT_BF16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2002_05814_b200 import build
    build.build()
    assert torch.cuda.is_available()


def _windows(elems, chunk_elems, rng, n_random=6, width=5000):
    width = min(width, elems)
    w = [(0, width), (elems - width, elems), (elems - 3, elems)]
    if elems > chunk_elems:
        last = (elems - 1) // chunk_elems * chunk_elems
        w += [(chunk_elems - 100, chunk_elems + 100), (last - 64, min(elems, last + 4096 + 64))]
    for _ in range(n_random):
        lo = int(rng.integers(0, elems - width + 1))
        w.append((lo, lo + width))
    return [(max(0, a), min(elems, b)) for a, b in w]


class Shadow:
    """The oracle fed with zero-stride placeholder arrays: schedules only, no object bytes."""

    def __init__(self, w: wl.Workload):
        self.o = OracleStore(w.chunk_bytes, w.degree, w.degree)
        self.ph = {}

    def placeholder(self, nbytes, dtype):
        key = (nbytes, dtype)
        if key not in self.ph:
            self.ph[key] = np.broadcast_to(np.zeros(1, np.float32 if dtype == DT_F32 else np.uint16), (nbytes // (4 if dtype == DT_F32 else 2),))
        return self.ph[key]


def _ctx(w, arena_bytes, **kw):
    arena = torch.empty(arena_bytes, dtype=torch.uint8, device="cuda")
    c = hpl.Context(w.chunk_bytes, w.degree, w.degree, arena=arena.data_ptr(), arena_bytes=arena_bytes,
                    stream=torch.cuda.current_stream().cuda_stream, **kw)
    return arena, c


def _check_reduce_windows(w, members_obj_at, seeds, out_f32: torch.Tensor, rng):
    chunk_elems = w.chunk_bytes // w.elem_bytes
    for lo, hi in _windows(w.elems, chunk_elems, rng):
        objs = {o: wl.values_np(w.dist, seeds[o], o, lo, hi - lo, w.dtype) for o in members_obj_at}
        want = ov.tree_reduce(members_obj_at, w.degree, objs)
        got = out_f32[lo:hi].cpu().numpy()
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (lo, hi)
        ref = ov.naive_sum_f64(members_obj_at, objs)
        err = np.max(np.abs(got.astype(np.float64) - ref)) / max(np.max(np.abs(ref)), 1e-30)
        assert err <= 1e-5 * math.ceil(math.log2(max(2, len(members_obj_at))))


def test_cfg2_broadcast_64mib_to_16_receivers():
    w = wl.workload("cfg2")
    S = w.object_bytes
    arena, c = _ctx(w, 64 << 20)
    sh = Shadow(w)
    src = wl.values_torch(w.dist, w.seed, 0, 0, w.elems, "f32")
    recv = [torch.zeros(w.elems, dtype=torch.float32, device="cuda") for _ in range(16)]
    c.create(0, 99, S)
    sh.o.create(0, 99, S, DT_F32)
    for j in range(16):
        c.create(1 + j, j, S)
        sh.o.create(1 + j, j, S, DT_F32)
    c.put(0, src.data_ptr(), S)
    sh.o.put(0, sh.placeholder(S, DT_F32), S)
    c.broadcast(0, list(range(1, 17)))
    sh.o.broadcast(0, list(range(1, 17)))
    offs = wl.uniform_offsets_ns(w.seed, 16, w.extra["join_window_ns"])
    for j in sorted(range(16), key=lambda j: (offs[j], j)):
        c.advance(offs[j])
        sh.o.advance(offs[j])
        c.join(1 + j, recv[j].data_ptr())
        sh.o.join(1 + j)
    for j in range(16):
        c.get(1 + j)
        sh.o.get(1 + j)
    assert c.schedule_dump(0) == sh.o.dump(0)
    rng = np.random.default_rng(0)
    for j in range(16):
        assert torch.equal(recv[j].view(torch.int32), src.view(torch.int32))       # every byte, compared on the device
    for lo, hi in _windows(w.elems, w.chunk_bytes // 4, rng):
        want = wl.values_np(w.dist, w.seed, 0, lo, hi - lo)
        for j in (0, 7, 15):
            assert recv[j][lo:hi].cpu().numpy().tobytes() == want.tobytes()
    st = c.stats()
    assert st["bytes_read_planned"] == S and st["bytes_written_planned"] == 16 * S
    c.shutdown()


def test_cfg3_fifty_rounds_first_8_of_16_gradients():
    """All 50 rounds of the async-SGD configuration, each with fresh object contents and fresh arrival times
    (seed = base + round).  The context and its arena are reused: every round ends with its Deletes."""
    w = wl.workload("cfg3")
    S = w.object_bytes
    arena, c = _ctx(w, (64 << 20) + 2 * S)
    rng = np.random.default_rng(1)
    t0 = 0
    for rnd in range(50):
        sh = Shadow(w)
        seeds = {i: w.seed + rnd for i in range(16)}          # contents are a function of (seed, object index)
        dev = [wl.values_torch(w.dist, seeds[i], i, 0, w.elems, "f32") for i in range(16)]
        t0 += 1_000_000_000
        c.advance(t0)
        sh.o.advance(t0)
        for i in range(16):
            c.create(i, i, S)
            sh.o.create(i, i, S, DT_F32)
        c.reduce(100, list(range(16)), 8)
        sh.o.reduce(100, list(range(16)), 8)
        arr = wl.exponential_arrivals_ns(w.seed + rnd, 16, w.extra["mean_arrival_ns"])
        for i in sorted(range(16), key=lambda i: (arr[i], i)):
            c.advance(t0 + arr[i])
            sh.o.advance(t0 + arr[i])
            c.put(i, dev[i].data_ptr(), S)
            sh.o.put(i, sh.placeholder(S, DT_F32), S)
        st0 = c.stats()
        ptr, n = c.get(100)
        assert n == w.elems * 4 and c.schedule_dump(100) == sh.o.dump(100)
        off = ptr - arena.data_ptr()
        out = arena[off:off + n].view(torch.float32)
        obj_at = sh.o.reduces[100]["sched"].obj_at
        assert sorted(obj_at) == sorted(sorted(range(16), key=lambda i: (arr[i], i))[:8])
        _check_reduce_windows(w, obj_at, seeds, out, rng)
        st = c.stats()
        assert st["kernel_launches"] - st0["kernel_launches"] == 1 and st["bytes_read_planned"] - st0["bytes_read_planned"] == 8 * S
        for i in [100] + list(range(16)):
            c.delete(i)
        del dev
    c.shutdown()


def test_cfg4_policy_round_bf16():
    w = wl.workload("cfg4")
    S = w.object_bytes
    arena, c = _ctx(w, (64 << 20) + w.elems * 4)
    sh = Shadow(w)
    policy = wl.values_torch(w.dist, w.seed + 1000, 1000, 0, w.elems, "bf16")
    recv = [torch.zeros(w.elems, dtype=torch.bfloat16, device="cuda") for _ in range(64)]
    c.create(5000, 900, S, hpl.HPL_BF16)
    sh.o.create(5000, 900, S, DT_BF16)
    c.put(5000, policy.data_ptr(), S)
    sh.o.put(5000, sh.placeholder(S, DT_BF16), S)
    dsts = [6000 + j for j in range(64)]
    for j, dd in enumerate(dsts):
        c.create(dd, 1000 + j, S, hpl.HPL_BF16)
        sh.o.create(dd, 1000 + j, S, DT_BF16)
    c.broadcast(5000, dsts)
    sh.o.broadcast(5000, dsts)
    for j, dd in enumerate(dsts):
        c.join(dd, recv[j].data_ptr())
        sh.o.join(dd)
    for dd in dsts:
        c.get(dd)
        sh.o.get(dd)
    assert c.schedule_dump(5000) == sh.o.dump(5000)
    for j in range(64):
        assert torch.equal(recv[j].view(torch.int16), policy.view(torch.int16))
    del recv
    c.advance(sh.o.now + 1)
    sh.o.advance(sh.o.now + 1)
    seeds = {i: w.seed + i for i in range(64)}
    dev = [wl.values_torch(w.dist, seeds[i], i, 0, w.elems, "bf16") for i in range(64)]
    for i in range(64):
        c.create(i, i, S, hpl.HPL_BF16)
        sh.o.create(i, i, S, DT_BF16)
        c.put(i, dev[i].data_ptr(), S)
        sh.o.put(i, sh.placeholder(S, DT_BF16), S)
    c.reduce(9000, list(range(64)), 64, hpl.HPL_SUM, hpl.HPL_BF16)
    sh.o.reduce(9000, list(range(64)), 64, 0, DT_BF16)
    ptr, n = c.get(9000)
    assert n == w.elems * 4 and c.schedule_dump(9000) == sh.o.dump(9000)
    off = ptr - arena.data_ptr()
    out = arena[off:off + n].view(torch.float32)
    _check_reduce_windows(w, sh.o.reduces[9000]["sched"].obj_at, seeds, out, np.random.default_rng(2))
    c.shutdown()


@pytest.mark.parametrize("size", [(1 << 10) << (2 * j) for j in range(11)])     # 1 KiB ... 1 GiB in powers of 4
def test_cfg5_fault_tolerant_reduce(size):
    w = wl.cfg5_at(size)
    S = w.object_bytes
    arena, c = _ctx(w, (64 << 20) + 8 * S)      # target + the partial results of the subtrees beside worker 7's root path
    sh = Shadow(w)
    seeds = {i: w.seed + i for i in range(32)}
    dev = [wl.values_torch(w.dist, seeds[i], i, 0, w.elems, "f32") for i in range(32)]
    C = wl.n_chunks(S, w.chunk_bytes)
    assert w.chunk_bytes == min(4 << 20, S)          # the configuration's own chunk: whole object if smaller
    h = int(0.4 * C)
    for i in range(32):
        c.create(i, i, S)
        sh.o.create(i, i, S, DT_F32)
    c.reduce(100, list(range(32)), 32)
    sh.o.reduce(100, list(range(32)), 32)
    for i in range(32):
        nb = S if i != 7 else h * w.chunk_bytes
        if nb:
            c.put(i, dev[i].data_ptr(), nb)
            sh.o.put(i, sh.placeholder(S, DT_F32), nb)
    c.progress()
    c.advance(1)
    sh.o.advance(1)
    c.fail(7)
    sh.o.fail(7)
    ptr, n = c.get(100)
    assert c.schedule_dump(100) == sh.o.dump(100)
    off = ptr - arena.data_ptr()
    out = arena[off:off + n].view(torch.float32)
    obj_at = sh.o.reduces[100]["sched"].obj_at
    assert sorted(obj_at) == [i for i in range(32) if i != 7]
    _check_reduce_windows(w, obj_at, seeds, out, np.random.default_rng(3))
    c.shutdown()


def test_objects_beyond_four_gib():
    """Byte offsets past 2^32 and element indices past 2^30: a Reduce over three 5 GiB objects with a ragged last chunk,
    its output broadcast to two receivers; windows around the 4 GiB mark and the tail against the oracle."""
    import dataclasses
    base = wl.workload("cfg3")
    elems = (5 << 30) // 4 + 1000
    w = dataclasses.replace(base, elems=elems, degree=2)
    S = w.object_bytes
    arena, c = _ctx(w, (64 << 20) + S)
    sh = Shadow(w)
    seeds = {i: w.seed + i for i in range(3)}
    dev = [wl.values_torch(w.dist, seeds[i], i, 0, elems, "f32") for i in range(3)]
    recv = [torch.zeros(elems, dtype=torch.float32, device="cuda") for _ in range(2)]
    for i in range(3):
        c.create(i, i, S)
        sh.o.create(i, i, S, DT_F32)
        c.put(i, dev[i].data_ptr(), S)
        sh.o.put(i, sh.placeholder(S, DT_F32), S)
    c.reduce(100, [0, 1, 2], 3)
    sh.o.reduce(100, [0, 1, 2], 3)
    for j in range(2):
        c.create(200 + j, 10 + j, S)
        sh.o.create(200 + j, 10 + j, S, DT_F32)
    c.broadcast(100, [200, 201])
    sh.o.broadcast(100, [200, 201])
    for j in range(2):
        c.join(200 + j, recv[j].data_ptr())
        sh.o.join(200 + j)
    ptr, n = c.get(100)
    for j in range(2):
        c.get(200 + j)
    assert n == S and c.schedule_dump(100) == sh.o.dump(100)
    off = ptr - arena.data_ptr()
    out = arena[off:off + n].view(torch.float32)
    obj_at = sh.o.reduces[100]["sched"].obj_at
    chunk_elems = w.chunk_bytes // 4
    mark = (1 << 32) // 4                                            # the element at byte offset 2^32
    for lo, hi in [(mark - 3000, mark + 3000), (elems - 5000, elems), (0, 5000),
                   ((elems - 1) // chunk_elems * chunk_elems - 64, elems)]:
        objs = {o: wl.values_np(w.dist, seeds[o], o, lo, hi - lo) for o in obj_at}
        want = ov.tree_reduce(obj_at, w.degree, objs)
        assert np.array_equal(out[lo:hi].cpu().numpy().view(np.uint32), want.view(np.uint32)), (lo, hi)
    for j in range(2):
        assert torch.equal(recv[j].view(torch.int32), out.view(torch.int32))
    c.shutdown()
