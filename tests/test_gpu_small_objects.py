"""Small objects (under 64 KiB, Section 3.2): many collectives requested together are served by shared waves.
Values must not care: every target and every receiver is compared with the oracle, bit for bit."""
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


@pytest.mark.parametrize("nbytes", [1 << 10, 4 << 10, 16 << 10, (64 << 10) - 4])
def test_thirty_two_small_reduces_in_one_pass(nbytes):
    elems = nbytes // 4
    p = Pair(min(nbytes, 16 << 10) // 16 * 16 or 16, 2, 2)
    oid = 0
    targets = []
    for r in range(32):
        k = 2 + r % 7
        ids = list(range(oid, oid + k))
        oid += k
        for i in ids:
            p.create(i, i, gen(("uniform",), 300 + r, i, elems))
            p.put(i)
        p.reduce(10_000 + r, ids, k, hpl.HPL_SUM if r % 5 else hpl.HPL_MAX)
        targets.append(10_000 + r)
    st0 = p.c.stats()
    for t in targets:
        p.check_target_bits(t)
        p.check_schedule(t)
    st = p.c.stats()
    assert st["reduce_launches"] - st0["reduce_launches"] <= 3        # 32 tasks in shared waves, not 32 launches
    p.close()


def test_small_composed_reduces_broadcasts_and_allreduce_in_one_pass():
    elems = 3000                                       # 12,000 bytes: two chunks of 8 KiB, ragged
    p = Pair(8 << 10, 2, 2)
    for i in range(12):
        p.create(i, i, gen(("uniform",), 310, i, elems))
    for i in range(12, 16):
        p.create(i, i, gen(("normal", 0.02), 311, i, elems, "bf16"))
    p.reduce(100, [0, 1, 2, 3], 4)
    p.reduce(101, [4, 5, 6], 3)
    p.reduce(102, [100, 101, 7], 3)                    # consumes two outputs of the same pass
    p.reduce(103, [12, 13, 14, 15], 4, 0, DT_BF16)      # bf16 inputs: another wave of the same pass
    p.reduce(104, [102, 8], 2)                         # a second level of composition
    for j in range(5):
        p.create(200 + j, 50 + j, nbytes=elems * 4, dtype=DT_F32)
    p.broadcast(104, [200, 201, 202])                  # reduce followed by broadcast
    p.broadcast(9, [203, 204])                         # a plain small broadcast
    for j in range(5):
        p.join(200 + j)
    p.advance(3)
    for i in range(16):
        p.put(i)
    for t in (104, 100, 101, 102, 103):
        p.check_target_bits(t)
    for j in range(5):
        p.check_receiver_bytes(200 + j)
    st = p.c.stats()
    assert st["kernel_launches"] <= 6 and st["fused_fanout_tasks"] == 1
    p.close()


def test_small_and_large_collectives_keep_their_order():
    p = Pair(64 << 10, 2, 2)
    for i in range(4):
        p.create(i, i, gen(("normal", 0.02), 320, i, 20_000, "bf16"))     # 40,000 bytes: small; the fp32 output is not
        p.put(i)
    for i in range(4, 6):
        p.create(i, i, gen(("uniform",), 321, i, 20_000))
        p.put(i)
    p.reduce(100, [0, 1, 2, 3], 4, 0, DT_BF16)
    p.reduce(101, [100, 4, 5], 3)                       # 80,000-byte objects: a launch of its own, after the small wave
    p.check_target_bits(101)
    p.check_target_bits(100)
    p.close()


def test_small_reduce_with_a_failure_and_a_spare():
    p = Pair(4096, 2, 2)
    for i in range(9):
        p.create(i, i, gen(("uniform",), 330, i, 1500))
    p.reduce(100, list(range(9)), 8)
    for i in range(8):
        p.advance(i + 1)
        p.put(i, 4096 if i == 3 else None)
    p.progress()
    p.advance(20)
    p.fail(3)
    p.advance(30)
    p.put(8)
    p.check_target_bits(100)
    p.check_schedule(100)
    p.close()


def _dag_timeline(seed):
    """Up to a dozen collectives, most on small objects, some consuming others' outputs, some broadcast, requested before
    any object exists; objects then arrive in random order (some partly, some never, some workers fail)."""
    rng = np.random.default_rng(seed)
    chunk = int(rng.choice([1024, 4096, 16384]))
    elems = int(rng.integers(1, 4)) * (chunk // 4) + int(rng.choice([0, 0, 8]))
    elems -= elems % 8
    big = rng.random() < 0.25                      # sometimes above the threshold: mixes shared and own launches
    if big:
        elems = 24 * 1024
    p = Pair(chunk, int(rng.integers(1, 5)), int(rng.integers(1, 3)), eager=bool(rng.random() < 0.25), fuse=bool(rng.random() < 0.7))
    n_ops = int(rng.integers(3, 12))
    oid, recv_id = 0, 5000
    outputs, plain, receivers = [], [], []
    def new_obj(bf):
        nonlocal oid
        i = oid
        oid += 1
        p.create(i, i, gen(("normal", 0.02), 800 + seed, i, elems, "bf16") if bf else gen(("uniform",), 800 + seed, i, elems))
        plain.append(i)
        return i
    for q in range(n_ops):
        bf = rng.random() < 0.3
        n_src = int(rng.integers(1, 6))
        srcs = [new_obj(bf) for _ in range(n_src)]
        if not bf and outputs and rng.random() < 0.6:       # consume earlier outputs (fp32)
            for o_ in rng.choice(outputs, size=min(len(outputs), int(rng.integers(1, 3))), replace=False):
                if int(o_) not in srcs:
                    srcs.append(int(o_))
        tgt = 1000 + q
        k = len(srcs) if rng.random() < 0.7 else int(rng.integers(1, len(srcs) + 1))
        p.reduce(tgt, srcs, k, 0, DT_BF16 if bf else DT_F32)
        outputs.append(tgt)
        if rng.random() < 0.4:
            dst = []
            for _ in range(int(rng.integers(1, 4))):
                p.create(recv_id, 900 + recv_id, nbytes=elems * 4, dtype=DT_F32)
                dst.append(recv_id)
                recv_id += 1
            p.broadcast(tgt, dst)
            receivers += dst
            for d_ in dst:
                if rng.random() < 0.8:
                    p.join(d_)
    t = 0
    for i in rng.permutation(plain):
        t += int(rng.integers(0, 5))
        p.advance(t)
        if rng.random() < 0.9 and p.o.objects[int(i)].alive:
            p.put(int(i), None if rng.random() < 0.8 else min(chunk, p.host[int(i)].nbytes))
        if rng.random() < 0.1:
            p.progress()
        if rng.random() < 0.05:
            p.fail(int(rng.choice(plain)))
    for oid_ in outputs + receivers:
        ro = OK
        try:
            want = p.o.get(oid_)
        except StoreError as e:
            ro = e.code
        rl, ptr, nb = p.c.try_get(oid_)
        assert rl == ro, (oid_, ro, rl)
        if ro == OK:
            assert p.view(ptr, nb).cpu().numpy().tobytes() == want.tobytes(), f"object {oid_} differs"
        t = max(t, p.o.now)
        p.advance(t)
    p.close()


@pytest.mark.parametrize("block", range(3))
def test_random_dags_of_small_collectives_match_the_oracle(block):
    for seed in range(block * 40, (block + 1) * 40):
        try:
            _dag_timeline(seed)
        except AssertionError as e:
            raise AssertionError(f"seed {seed}: {e}") from e
