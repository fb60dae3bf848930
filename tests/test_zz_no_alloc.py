"""hpl_reduce_noalloc -- the reduce entry point for callers that may not allocate device memory
(allocator callbacks, serving loops with a frozen memory map).  It keeps its scratch in a fixed array
inside the library, shared by all calls, so the test calls it twice in a row with different inputs
and compares each result, bit for bit, with what the ordinary hpl_reduce path gives for the same
objects arriving in the same order -- and with the oracle's evaluation of the same tree."""
import numpy as np
import pytest
import torch

import paper_2002_05814_b200 as hpl
from oracle import reduce_tree as ort
from oracle import values as ov
from oracle.store import DT_F32, DT_BF16
from tests.harness import Pair, gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2002_05814_b200 import build
    build.build()
    assert torch.cuda.is_available()


def _existing_path(objs, degree, dtype, op):
    """Result of hpl_put x n + hpl_reduce + hpl_get for the same objects, as device tensors."""
    p = Pair(64 << 10, degree)
    for i, a in enumerate(objs):
        p.create(i, i, a)
        p.advance(i + 1)
        p.put(i)
    p.reduce(1000, list(range(len(objs))), len(objs), op, dtype)
    ptr, n = p.c.get(1000)
    want = p.view(ptr, n).view(torch.float32).clone()
    dev = [p.dev[i] for i in range(len(objs))]
    p.close()
    return dev, want


@pytest.mark.parametrize("dtype,n,degree,elems", [("f32", 8, 2, 100_003), ("bf16", 64, 4, 40_000), ("f32", 3, 1, 5)])
def test_two_calls_in_a_row_match_the_existing_entry_point(dtype, n, degree, elems):
    code = DT_BF16 if dtype == "bf16" else DT_F32
    stream = torch.cuda.current_stream().cuda_stream
    for call, (seed, op) in enumerate(((41, hpl.HPL_SUM), (42, hpl.HPL_MAX if dtype == "f32" else hpl.HPL_SUM))):
        m = n if call == 0 else max(1, n - 1)            # the second call has another shape: the scratch is rewritten
        objs = [gen(("uniform",) if dtype == "f32" else ("normal", 0.02), seed, i, elems, dtype) for i in range(m)]
        dev, want = _existing_path(objs, degree, code, op)
        out = torch.full((elems,), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        if call == 1:      # the first call on a device looks the scratch array's address up; from then on nothing may change
            free0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
        rc = hpl.reduce_noalloc([t.data_ptr() for t in dev], degree, op, code, elems, out.data_ptr(), stream)
        assert rc == hpl.HPL_OK
        torch.cuda.synchronize()
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_reserved() == reserved0, "device memory was allocated"
        assert torch.equal(out.view(torch.int32), want.view(torch.int32))
        # ... and the oracle's evaluation of the tree these arrivals form (objects arrive in index order)
        sched = ort.ReduceSchedule(list(range(m)), m, degree)
        for i in range(m):
            sched.on_arrival(i)
        ref = ov.tree_reduce(sched.obj_at, degree, dict(enumerate(objs)), op)
        assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))


def test_sizes_beyond_the_fixed_scratch_are_refused():
    x = torch.zeros(16, device="cuda")
    out = torch.zeros(16, device="cuda")
    too_many = [x.data_ptr()] * 257
    assert hpl.reduce_noalloc(too_many, 2, hpl.HPL_SUM, DT_F32, 16, out.data_ptr()) == hpl.HPL_ERR_INVALID
    assert hpl.reduce_noalloc([x.data_ptr()], 2, hpl.HPL_SUM, DT_F32, (1 << 32) + 1, out.data_ptr()) == hpl.HPL_ERR_INVALID
    assert hpl.reduce_noalloc([x.data_ptr() + 4], 2, hpl.HPL_SUM, DT_F32, 4, out.data_ptr()) == hpl.HPL_ERR_INVALID
    torch.cuda.synchronize()
    assert float(out.abs().sum()) == 0.0
