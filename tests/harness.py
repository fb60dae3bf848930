"""Drives the CUDA library and the oracle with the same seeded inputs and events (GPU tests only)."""
from __future__ import annotations

import numpy as np
import torch

import paper_2002_05814_b200 as hpl
import workloads as wl
from oracle.store import OracleStore, DT_F32, DT_BF16


def to_device(a: np.ndarray) -> torch.Tensor:
    """float32 array, or uint16 bf16 bit patterns -> device tensor of the same bits."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


class Pair:
    def __init__(self, chunk_bytes, d_reduce=2, d_bcast=2, tau=0, arena_bytes=256 << 20, **flags):
        self.arena = torch.empty(arena_bytes, dtype=torch.uint8, device="cuda")
        self.stream = torch.cuda.current_stream().cuda_stream
        flags.setdefault("debug_guard_bytes", 256)      # canaries behind every block the library takes from the arena
        self.c = hpl.Context(chunk_bytes, d_reduce, d_bcast, arena=self.arena.data_ptr(), arena_bytes=arena_bytes,
                             stream=self.stream, virt_chunk_ns=tau, **flags)
        self.o = OracleStore(chunk_bytes, d_reduce, d_bcast, tau, flags.get("model_latency_ns", 0), flags.get("model_bandwidth_bps", 0))
        self.host: dict[int, np.ndarray] = {}
        self.dev: dict[int, torch.Tensor] = {}
        self.guarded: dict[int, torch.Tensor] = {}

    GUARD = 256   # bytes of canary before and after every receiver buffer

    def close(self):
        """Shuts the context down and checks what no test may violate: objects are immutable (the bytes of every
        put object are unchanged) and nothing was written outside a receiver's buffer or behind a block of the
        library's arena (targets, partial results, store copies of host objects)."""
        assert self.c.check_guards() == 0, "write behind an arena block"
        assert self.c.stats()["bounds_errors"] == 0, "a tile outside its object (bounds-checking build)"
        self.c.shutdown()
        torch.cuda.synchronize()
        for oid, a in self.host.items():
            got = self.dev[oid].view(torch.uint8).cpu().numpy().tobytes() if oid in self.dev else None
            assert got is None or got == a.tobytes(), f"object {oid} was modified"
        for oid, (whole, nbytes) in self.guarded.items():
            g = self.GUARD
            assert bool((whole[:g] == 0x5C).all()) and bool((whole[g + nbytes:] == 0x5C).all()), f"write outside receiver {oid}"

    def advance(self, t):
        self.c.advance(t)
        self.o.advance(t)

    def create(self, oid, worker, data: np.ndarray | None = None, nbytes=None, dtype=None):
        """A put object when ``data`` is given, else a receiver buffer of ``nbytes``."""
        if data is not None:
            dt = DT_BF16 if data.dtype == np.uint16 else DT_F32
            self.host[oid] = data
            self.dev[oid] = to_device(data)
            nbytes = data.nbytes
        else:
            dt = dtype
            pad = (-nbytes) % 16                       # keep the trailing canary 16-byte aligned after the buffer
            whole = torch.full((nbytes + pad + 2 * self.GUARD,), 0x5C, dtype=torch.uint8, device="cuda")
            whole[self.GUARD:self.GUARD + nbytes] = 0xA5
            self.guarded[oid] = (whole, nbytes)
            self.dev[oid] = whole[self.GUARD:self.GUARD + nbytes]
        self.c.create(oid, worker, nbytes, dt)
        self.o.create(oid, worker, nbytes, dt)

    def put(self, oid, nbytes=None):
        nbytes = self.host[oid].nbytes if nbytes is None else nbytes
        self.c.put(oid, self.dev[oid].data_ptr(), nbytes)
        self.o.put(oid, self.host[oid], nbytes)

    def reduce(self, target, srcs, k, op=0, dtype=DT_F32):
        self.c.reduce(target, srcs, k, op, dtype)
        self.o.reduce(target, srcs, k, op, dtype)

    def broadcast(self, src, dsts):
        self.c.broadcast(src, dsts)
        self.o.broadcast(src, dsts)

    def join(self, dst):
        self.c.join(dst, self.dev[dst].data_ptr())
        self.o.join(dst)

    def fail(self, worker):
        self.c.fail(worker)
        self.o.fail(worker)

    def progress(self):
        self.c.progress()

    def delete(self, oid):
        self.c.delete(oid)
        self.o.delete(oid)

    def view(self, ptr, nbytes) -> torch.Tensor:
        """Bytes at a device pointer that lies in the arena or in one of the buffers given to the library."""
        base = self.arena.data_ptr()
        if base <= ptr < base + self.arena.numel():
            return self.arena[ptr - base: ptr - base + nbytes]
        for t in self.dev.values():
            if t.data_ptr() == ptr:
                return t.view(torch.uint8)[:nbytes]
        raise AssertionError("pointer outside every known buffer")

    def check_schedule(self, op_id):
        assert self.c.schedule_dump(op_id) == self.o.dump(op_id)

    def check_target_bits(self, target):
        ptr, n = self.c.get(target)
        got = self.view(ptr, n).cpu().numpy().view(np.uint32)
        want = self.o.get(target).view(np.uint32)
        assert got.shape == want.shape
        bad = np.flatnonzero(got != want)
        assert bad.size == 0, f"{bad.size} of {got.size} words differ, first at {bad[:5]}"
        return self.view(ptr, n).view(torch.float32)

    def check_receiver_bytes(self, dst):
        ptr, n = self.c.get(dst)
        assert ptr == self.dev[dst].data_ptr()
        got = self.dev[dst].view(torch.uint8)[:n].cpu().numpy().tobytes()
        want = self.o.get(dst).tobytes()
        assert got == want


def gen(dist, seed, obj, elems, dtype="f32"):
    return wl.values_np(dist, seed, obj, 0, elems, dtype)
