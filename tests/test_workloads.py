"""The seeded input generators: host and device spellings agree, and the shapes are as stated."""
import numpy as np
import pytest
import torch

import workloads as wl


def test_scalar_and_numpy_hash_agree():
    a = wl._bits32_np(7, 3, 1000, 50, 1)
    assert [int(x) for x in a] == [wl.bits32_scalar(7, 3, 1000 + i, 1) for i in range(50)]


@pytest.mark.parametrize("dist,dtype", [(("uniform",), "f32"), (("normal", 1e-3), "f32"),
                                        (("normal", 0.02), "bf16"), (("smallint", 100), "f32")])
def test_host_and_torch_spellings_are_bit_identical(dist, dtype):
    a = wl.values_np(dist, wl.BASE_SEED, 5, 123, 70_000, dtype)
    t = wl.values_torch(dist, wl.BASE_SEED, 5, 123, 70_000, dtype, device="cpu", slab=1 << 14)
    if dtype == "bf16":
        tb = t.view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(a, tb)
    else:
        assert np.array_equal(a.view(np.uint32), t.numpy().view(np.uint32))


def test_distributions_have_the_stated_shape():
    u = wl.values_np(("uniform",), 1, 0, 0, 1 << 18)
    assert u.min() >= -1.0 and u.max() < 1.0 and abs(u.mean()) < 0.01 and abs(u.std() - 3 ** -0.5) < 0.01
    g = wl.values_np(("normal", 1e-3), 1, 0, 0, 1 << 18)
    assert abs(g.mean()) < 2e-5 and abs(g.std() / 1e-3 - 1) < 0.01
    # different objects and seeds decorrelate
    h = wl.values_np(("uniform",), 1, 1, 0, 1 << 18)
    assert abs(np.corrcoef(u, h)[0, 1]) < 0.01
    # a window is the same whatever the start of the request
    assert np.array_equal(u[1000:1100], wl.values_np(("uniform",), 1, 0, 1000, 100))


def test_bf16_rounding_matches_torch():
    x = np.random.default_rng(0).normal(0, 0.02, 100_000).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(wl.f32_to_bf16_bits(x), want)
    assert np.array_equal(wl.bf16_bits_to_f32(want), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_timelines():
    j = wl.uniform_offsets_ns(3, 1000)
    assert min(j) >= 0 and max(j) < 1_000_000 and abs(np.mean(j) - 5e5) < 3e4
    a = wl.exponential_arrivals_ns(3, 4000)
    assert min(a) >= 0 and abs(np.mean(a) / 5e6 - 1) < 0.06
    ev = wl.sort_events([(5, wl.EV_JOIN, 2), (5, wl.EV_FAIL, 9), (1, wl.EV_PUT, 3), (5, wl.EV_PUT, 1)])
    assert ev == [(1, wl.EV_PUT, 3), (5, wl.EV_FAIL, 9), (5, wl.EV_PUT, 1), (5, wl.EV_JOIN, 2)]


def test_workload_table():
    w = wl.workload("cfg3")
    assert w.object_bytes == 102_228_128 and wl.n_chunks(w.object_bytes, w.chunk_bytes) == 25
    assert w.object_bytes - 24 * w.chunk_bytes == 1_564_832
    assert wl.workload("cfg4").object_bytes == 64 * wl.MiB
    sizes = wl.workload("cfg5").extra["sizes_bytes"]
    assert sizes[0] == 1024 and sizes[-1] == wl.GiB and len(sizes) == 11
