"""Worker-per-GPU mode, values: the ranks are emulated as several contexts in ONE process on one GPU -- each with an
arena of its own, "peer" addresses being ordinary device addresses -- and driven level by level in turn, so no kernel
ever waits for another one.  Every rank runs only the tasks it owns; the results must equal the oracle's bit for bit."""
import numpy as np
import pytest
import torch

import paper_2002_05814_b200 as hpl
from oracle.store import OracleStore, DT_F32, DT_BF16
from tests.harness import to_device, gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2002_05814_b200 import build
    build.build()
    assert torch.cuda.is_available()


class Ranks:
    def __init__(self, world, chunk, d, fuse, arena_bytes=48 << 20, pipeline_chunks=0):
        self.world = world
        self.arenas = [torch.empty(arena_bytes, dtype=torch.uint8, device="cuda") for _ in range(world)]
        stream = torch.cuda.current_stream().cuda_stream
        self.c = [hpl.Context(chunk, d, d, arena=self.arenas[r].data_ptr(), arena_bytes=arena_bytes, stream=stream, fuse=fuse,
                              rank=r, world_size=world, debug_guard_bytes=256, pipeline_chunks=pipeline_chunks) for r in range(world)]
        for r in range(world):
            for q in range(world):
                if q != r:
                    self.c[r].set_peer_arena(q, self.arenas[q].data_ptr())
        self.live = list(range(world))
        self.o = OracleStore(chunk, d, d)
        self.host, self.dev = {}, {}
        self.plans = []              # levels of every plan that had any

    def each(self, name, *args):
        for r in self.live:
            getattr(self.c[r], name)(*args)

    def advance(self, t):
        self.each("advance", t)
        self.o.advance(t)

    def create(self, oid, worker, data=None, nbytes=None, dtype=DT_F32):
        if data is not None:
            self.host[oid] = data
            self.dev[oid] = to_device(data)
            nbytes, dtype = data.nbytes, (DT_BF16 if data.dtype == np.uint16 else DT_F32)
        else:
            self.dev[oid] = torch.full((nbytes,), 0xA5, dtype=torch.uint8, device="cuda")
        self.each("create", oid, worker, nbytes, dtype)
        self.o.create(oid, worker, nbytes, dtype)

    def put(self, oid, nbytes=None):
        nbytes = self.host[oid].nbytes if nbytes is None else nbytes
        self.each("put", oid, self.dev[oid].data_ptr(), nbytes)
        self.o.put(oid, self.host[oid], nbytes)

    def reduce(self, target, srcs, k, dtype=DT_F32):
        self.each("reduce", target, srcs, k, 0, dtype)
        self.o.reduce(target, srcs, k, 0, dtype)

    def broadcast(self, src, dsts):
        self.each("broadcast", src, dsts)
        self.o.broadcast(src, dsts)

    def join(self, dst):
        self.each("join", dst, self.dev[dst].data_ptr())
        self.o.join(dst)

    def fail_rank(self, rank):
        self.live.remove(rank)
        self.each("fail_rank", rank)
        for w in sorted({e.worker for e in self.o.objects.values() if e.alive and e.worker >= 0 and e.worker % self.world == rank}):
            self.o.fail(w)

    def drive(self):
        while True:
            self.each("progress")
            n = {self.c[r].pending_levels() for r in self.live}
            assert len(n) == 1, "the ranks' plans differ"
            n = n.pop()
            if n == 0:
                return
            self.plans.append(n)
            for _ in range(n):
                self.each("run_level")
                for r in self.live:
                    assert self.c[r].sync() == hpl.HPL_OK
                # (here every rank would run its barrier)

    def target_bits(self, target):
        ptrs = {self.c[r].get(target) for r in self.live}
        assert len(ptrs) == 1                                # peer addresses are plain addresses in this emulation
        ptr, n = ptrs.pop()
        home = target % self.world
        off = ptr - self.arenas[home].data_ptr()
        assert 0 <= off < self.arenas[home].numel(), "the output does not live on rank target % world"
        return self.arenas[home][off:off + n].cpu().numpy().view(np.uint32)

    def close(self):
        for r in range(self.world):
            if r in self.live:
                assert self.c[r].check_guards() == 0
            self.c[r].shutdown()
        for oid, a in self.host.items():
            assert self.dev[oid].view(torch.uint8).cpu().numpy().tobytes() == a.tobytes()


@pytest.mark.parametrize("world,fuse,dtype", [(2, False, "f32"), (4, False, "f32"), (4, True, "f32"), (3, False, "bf16"), (8, False, "f32")])
def test_tree_reduce_across_ranks_matches_the_oracle(world, fuse, dtype):
    elems, chunk, k = 9 * 4096 + 11, 16 << 10, 8
    p = Ranks(world, chunk, 2, fuse)
    for i in range(k):
        p.create(i, i, gen(("uniform",) if dtype == "f32" else ("normal", 0.02), 400, i, elems, dtype))
    p.reduce(100, list(range(k)), k, DT_BF16 if dtype == "bf16" else DT_F32)
    for i in range(k):
        p.advance(i + 1)
        p.put(i, None if i != 3 else 2 * chunk)              # a member that is only partly there at first
    p.drive()
    p.advance(50)
    p.put(3)
    p.drive()
    assert np.array_equal(p.target_bits(100), p.o.get(100).view(np.uint32))
    for r in p.live:
        assert p.c[r].schedule_dump(100) == p.o.dump(100)
    st = [p.c[r].stats() for r in range(world)]
    assert sum(s["reduce_tasks"] > 0 for s in st) >= min(2, world)        # the work is spread over the ranks
    if not fuse:
        assert sum(s["bytes_written_planned"] for s in st) >= 4 * elems * 4   # every internal node wrote its result
    p.close()


def test_broadcast_follows_the_tree_across_ranks_and_allreduce_is_fused_at_the_root():
    elems, chunk, R = 6 * 4096 + 5, 16 << 10, 6
    p = Ranks(4, chunk, 2, False)
    for i in range(4):
        p.create(i, i, gen(("uniform",), 401, i, elems))
    src = gen(("uniform",), 402, 9, elems)
    p.create(9, 2, src)
    for j in range(R):
        p.create(50 + j, 10 + j, nbytes=elems * 4)
        p.create(70 + j, 20 + j, nbytes=elems * 4)
    p.reduce(100, [0, 1, 2, 3], 4)
    p.broadcast(100, [50 + j for j in range(R)])               # reduce followed by broadcast
    p.broadcast(9, [70 + j for j in range(R)])                 # a plain object: two send slots per copy, depth > 1
    p.put(9)
    for j in range(R):
        p.advance(j + 1)
        p.join(50 + j)
        p.join(70 + j)
    p.advance(20)
    for i in range(4):
        p.put(i)
    p.drive()
    want = p.o.get(100)
    assert np.array_equal(p.target_bits(100), want.view(np.uint32))
    for j in range(R):
        for r in p.live:
            p.c[r].get(50 + j)
            p.c[r].get(70 + j)
        assert p.dev[50 + j].cpu().numpy().tobytes() == p.o.get(50 + j).tobytes() == want.tobytes()
        assert p.dev[70 + j].cpu().numpy().tobytes() == src.tobytes()
    assert p.c[0].schedule_dump(9) == p.o.dump(9)
    p.close()


def test_a_rank_is_lost_between_plans_and_the_survivors_sum_is_exact():
    elems, chunk, k = 5 * 4096 + 3, 16 << 10, 8
    p = Ranks(4, chunk, 2, False)
    for i in range(k):
        p.create(i, i, gen(("uniform",), 403, i, elems))
    p.reduce(100, list(range(k)), k)
    for i in range(k):
        p.advance(i + 1)
        p.put(i, None if i != 6 else chunk)
    p.drive()                                                 # partial results exist on every rank
    p.advance(30)
    p.fail_rank(3)                                            # workers 3 and 7 and what the library kept on that GPU
    p.advance(40)
    p.put(6)
    p.drive()
    got = p.target_bits(100)
    assert np.array_equal(got, p.o.get(100).view(np.uint32))
    ref = sum(p.host[i].astype(np.float64) for i in (0, 1, 2, 4, 5, 6))
    assert np.max(np.abs(got.view(np.float32) - ref)) / np.max(np.abs(ref)) <= 3e-5
    for r in p.live:
        assert p.c[r].schedule_dump(100) == p.o.dump(100)
    p.close()


@pytest.mark.parametrize("world,pieces", [(4, 2), (2, 1), (8, 3)])
def test_pieces_of_a_chunk_range_move_up_the_tree_one_level_apart(world, pieces):
    """pipeline_chunks: while a tree level reduces piece j, the level above it reduces piece j - 1 (Section 3.3).  The plan
    has tree height + pieces - 1 levels instead of tree height; the bits are the same."""
    elems, chunk, k = 12 * 4096, 16 << 10, 8                   # 12 chunks
    p = Ranks(world, chunk, 2, False, pipeline_chunks=pieces)
    for i in range(k):
        p.create(i, i, gen(("uniform",), 410, i, elems))
    p.reduce(100, list(range(k)), k)
    for i in range(k):
        p.advance(i + 1)
        p.put(i)
    p.drive()
    assert np.array_equal(p.target_bits(100), p.o.get(100).view(np.uint32))
    n_pieces = -(-12 // pieces)
    assert p.plans == [3 + n_pieces - 1]                        # the tree of 8 has three levels of internal nodes
    p.close()


def test_a_broadcast_chain_is_pipelined_hop_by_hop_within_one_plan():
    elems, chunk, R = 6 * 4096, 16 << 10, 5                     # 6 chunks, one send slot per copy: a chain of 5 hops
    p = Ranks(3, chunk, 1, False, pipeline_chunks=1)
    src = gen(("uniform",), 411, 0, elems)
    p.create(0, 0, src)
    for j in range(R):
        p.create(10 + j, 1 + j, nbytes=elems * 4)
    p.put(0)
    p.broadcast(0, [10 + j for j in range(R)])
    for j in range(R):
        p.advance(j + 1)                                        # each joins while its predecessor is still receiving
        p.join(10 + j)
    p.drive()
    for j in range(R):
        for r in p.live:
            p.c[r].get(10 + j)
        assert p.dev[10 + j].cpu().numpy().tobytes() == src.tobytes() == p.o.get(10 + j).tobytes()
    assert p.c[0].schedule_dump(0) == p.o.dump(0)
    assert p.plans == [R + 6 - 1]                               # hop h works on piece j while hop h + 1 works on piece j - 1
    p.close()


def _rank_timeline(seed):
    """A random timeline on emulated ranks: instalment Puts, joins, worker failures, a lost rank, drives in between."""
    from oracle.store import StoreError, OK
    rng = np.random.default_rng(seed)
    world = int(rng.integers(2, 5))
    k, R = int(rng.integers(2, 9)), int(rng.integers(1, 5))
    kk = int(rng.integers(1, k + 1))
    d = int(rng.integers(1, 4))
    chunk = int(rng.choice([4096, 16384]))
    elems = int(rng.integers(1, 6)) * (chunk // 4) + int(rng.choice([0, 0, 3, 1000]))
    p = Ranks(world, chunk, d, bool(rng.random() < 0.5), arena_bytes=16 << 20, pipeline_chunks=int(rng.choice([0, 0, 1, 2])))
    T = 1000 - 1000 % world                                     # the output lives on rank 0, which is never lost here
    nbytes = elems * 4
    for i in range(k):
        p.create(i, int(rng.integers(0, 2 * world)), gen(("smallint", 30) if seed % 2 else ("uniform",), 600 + seed, i, elems))
    for j in range(R):
        p.create(500 + j, int(rng.integers(0, 2 * world)), nbytes=nbytes)
    p.reduce(T, list(range(k)), kk)
    p.broadcast(T, [500 + j for j in range(R)])
    prefix = {i: 0 for i in range(k)}
    joiners = [500 + j for j in range(R)]
    lost_rank = False
    t = 0
    for _ in range(int(rng.integers(2 * k, 5 * k + 6))):
        t = max(t + int(rng.integers(0, 40)), p.o.now)
        p.advance(t)
        r = rng.random()
        if r < 0.5:
            i = int(rng.integers(0, k))
            if p.o.objects[i].alive:
                nb_ = nbytes if rng.random() < 0.5 else min(nbytes, prefix[i] + chunk)
                p.put(i, nb_)
                prefix[i] = nb_
        elif r < 0.58:
            w = int(rng.integers(0, 2 * world))
            p.each("fail", w)
            p.o.fail(w)
        elif r < 0.63 and not lost_rank and world > 2:
            p.fail_rank(int(rng.integers(1, world)))             # never rank 0, where the output lives
            lost_rank = True
        elif r < 0.75 and joiners:
            j = joiners.pop(0)
            if p.o.objects[j].alive:
                p.join(j)
        else:
            p.drive()
        for rk in p.live:
            assert p.c[rk].schedule_dump(T) == p.o.dump(T), "schedules differ"
    for i in range(k):
        if p.o.objects[i].alive:
            t = max(t + 5, p.o.now)
            p.advance(t)
            p.put(i)
    p.drive()
    for oid in [T] + [500 + j for j in range(R)]:
        ro, want = OK, None
        try:
            want = p.o.get(oid)
        except StoreError as e:
            ro = e.code
        codes = {p.c[rk].try_get(oid)[0] for rk in p.live}
        assert codes == {ro}, (oid, ro, codes)
        if ro == OK:
            got = p.target_bits(T).tobytes() if oid == T else p.dev[oid].cpu().numpy().tobytes()
            assert got == want.tobytes(), f"object {oid} differs"
    p.close()


def test_pieces_are_counted_from_the_objects_first_chunk_not_the_tasks():
    """A timeline that once gave wrong bits: tasks of one tree covered different chunk ranges, and a parent's piece was
    released in the same level as the child's."""
    _rank_timeline(1111)


@pytest.mark.parametrize("block", range(4))
def test_random_timelines_on_emulated_ranks_match_the_oracle(block):
    for seed in range(block * 30, (block + 1) * 30):
        try:
            _rank_timeline(seed)
        except AssertionError as e:
            raise AssertionError(f"seed {seed}: {e}") from e


def _rank_timeline_composed(seed):
    """As above with more of the path: a bf16 or fp32 Reduce whose output feeds a second Reduce whose output is broadcast, and
    a plain object broadcast through its own tree.  A worker or a rank is taken out only after the pending levels have been
    driven (in this mode bytes move when the caller drives; what a copy could still serve must have moved before it goes)."""
    from oracle.store import StoreError, OK
    rng = np.random.default_rng(seed)
    world = int(rng.integers(2, 5))
    k, kb, R = int(rng.integers(2, 8)), int(rng.integers(1, 4)), int(rng.integers(1, 5))
    d = int(rng.integers(1, 4))
    chunk = int(rng.choice([4096, 16384]))
    elems = int(rng.integers(1, 6)) * (chunk // 4) + int(rng.choice([0, 0, 8, 1000]))
    elems -= elems % 8
    bf = bool(rng.random() < 0.35)
    p = Ranks(world, chunk, d, bool(rng.random() < 0.5), arena_bytes=16 << 20, pipeline_chunks=int(rng.choice([0, 0, 1, 2, 3])))
    T = 1000 - 1000 % world                                     # both outputs live on rank 0, which is never lost here
    B = T + world
    nbytes = elems * 4
    for i in range(k):
        p.create(i, int(rng.integers(0, 2 * world)),
                 gen(("normal", 0.02), 650 + seed, i, elems, "bf16") if bf else gen(("uniform",), 650 + seed, i, elems))
    for i in range(k, k + kb):
        p.create(i, int(rng.integers(0, 2 * world)), gen(("uniform",), 650 + seed, i, elems))
    X = k + kb
    p.create(X, int(rng.integers(0, 2 * world)), gen(("uniform",), 650 + seed, X, elems))
    for j in range(R):
        p.create(500 + j, int(rng.integers(0, 2 * world)), nbytes=nbytes)
        p.create(600 + j, int(rng.integers(0, 2 * world)), nbytes=nbytes)
    n_all = X + 1
    p.reduce(T, list(range(k)), int(rng.integers(1, k + 1)), DT_BF16 if bf else DT_F32)
    p.reduce(B, [T] + list(range(k, k + kb)), int(rng.integers(1, kb + 2)))
    p.broadcast(B, [500 + j for j in range(R)])
    p.broadcast(X, [600 + j for j in range(R)])
    size = {i: p.host[i].nbytes for i in range(n_all)}
    prefix = {i: 0 for i in range(n_all)}
    joiners = [500 + j for j in range(R)] + [600 + j for j in range(R)]
    rng.shuffle(joiners)
    lost_rank = False
    t = 0
    for _ in range(int(rng.integers(2 * n_all, 5 * n_all + 6))):
        t = max(t + int(rng.integers(0, 40)), p.o.now)
        p.advance(t)
        r = rng.random()
        if r < 0.5:
            i = int(rng.integers(0, n_all))
            if p.o.objects[i].alive:
                nb_ = size[i] if rng.random() < 0.5 else min(size[i], prefix[i] + chunk)
                p.put(i, nb_)
                prefix[i] = nb_
        elif r < 0.57:
            w = int(rng.integers(0, 2 * world))
            p.drive()
            p.each("fail", w)
            p.o.fail(w)
        elif r < 0.62 and not lost_rank and world > 2:
            p.drive()
            p.fail_rank(int(rng.integers(1, world)))
            lost_rank = True
        elif r < 0.78 and joiners:
            j = joiners.pop(0)
            if p.o.objects[j].alive:
                p.join(j)
        else:
            p.drive()
        for rk in p.live:
            assert p.c[rk].schedule_dump(T) == p.o.dump(T) and p.c[rk].schedule_dump(B) == p.o.dump(B), "schedules differ"
    for i in range(n_all):
        if p.o.objects[i].alive:
            t = max(t + 5, p.o.now)
            p.advance(t)
            p.put(i)
    p.drive()
    for oid in [T, B] + [500 + j for j in range(R)] + [600 + j for j in range(R)]:
        ro, want = OK, None
        try:
            want = p.o.get(oid)
        except StoreError as e:
            ro = e.code
        codes = {p.c[rk].try_get(oid)[0] for rk in p.live}
        assert codes == {ro}, (oid, ro, codes)
        if ro == OK:
            got = p.target_bits(oid).tobytes() if oid in (T, B) else p.dev[oid].cpu().numpy().tobytes()
            assert got == want.tobytes(), f"object {oid} differs"
    p.close()


@pytest.mark.parametrize("block", range(3))
def test_random_composed_timelines_on_emulated_ranks_match_the_oracle(block):
    for seed in range(block * 30, (block + 1) * 30):
        try:
            _rank_timeline_composed(seed)
        except AssertionError as e:
            raise AssertionError(f"seed {seed}: {e}") from e
