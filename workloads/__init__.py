"""Seeded synthetic inputs and arrival timelines for the reduce / broadcast workloads.

This module serves both the CPU oracle's tests and the CUDA path's tests and benchmark.
It holds none of the method's arithmetic: it only produces object contents (as a pure
function of ``(seed, object, element index)``) and event times.  Object contents exist
in two spellings of the same integer recipe -- numpy for the host and torch for the
device -- which must agree bit for bit (``tests/test_workloads.py`` checks that).

Recipe (all integer, so both spellings are exact):

* ``bits32(seed, obj, idx, lane)``: a 32-bit counter hash.  The key
  ``idx + seed*K_SEED + obj*K_OBJ + lane*K_LANE`` (mod 2^32) goes through three
  xorshift-multiply rounds with odd multipliers.
* ``uniform``: the top 24 bits ``u`` give ``(u - 2^23) / 2^23`` in [-1, 1): exact in fp32.
* ``normal(sigma)``: the four 16-bit halves of two hash lanes are added (an Irwin-Hall
  sum of four uniforms: bell shaped, mean 131070, standard deviation 37837.2..., support
  +-3.46 sigma); the centred integer (exact in fp32) is multiplied once, in fp32, by
  ``fp32(sigma / 37837.2...)``.  This stands in for N(0, sigma) without transcendental
  functions, whose last bit differs between host and device maths libraries.
* ``bf16``: the fp32 value rounded to nearest-even bf16 (host spelling returns the 16-bit
  patterns as uint16).

Timelines are plain Python integers (nanoseconds), generated on the host for both sides.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20020581

_M32 = 0xFFFFFFFF
_K_SEED = 0x9E3779B1
_K_OBJ = 0x6A09E667
_K_LANE = 0x3C6EF373
_MUL1 = 0xBB67AE85
_MUL2 = 0xA54FF53B
_MUL3 = 0x510E527F
_IH4_MEAN = 131070  # 4 * 65535 / 2
_IH4_STD = math.sqrt(4.0 * (65536.0 ** 2 - 1.0) / 12.0)

MiB = 1 << 20
KiB = 1 << 10
GiB = 1 << 30


# --------------------------------------------------------------------------- hash
def _key(seed: int, obj: int, lane: int) -> int:
    return (seed * _K_SEED + obj * _K_OBJ + lane * _K_LANE) & _M32


def _bits32_np(seed: int, obj: int, start: int, count: int, lane: int) -> np.ndarray:
    x = np.arange(start, start + count, dtype=np.uint64)
    x = (x + np.uint64(_key(seed, obj, lane))) & np.uint64(_M32)
    x ^= x >> np.uint64(15)
    x = (x * np.uint64(_MUL1)) & np.uint64(_M32)
    x ^= x >> np.uint64(13)
    x = (x * np.uint64(_MUL2)) & np.uint64(_M32)
    x ^= x >> np.uint64(16)
    x = (x * np.uint64(_MUL3)) & np.uint64(_M32)
    x ^= x >> np.uint64(14)
    return x


def _bits32_torch(seed: int, obj: int, start: int, count: int, lane: int, device):
    import torch

    x = torch.arange(start, start + count, dtype=torch.int64, device=device)
    x = (x + _key(seed, obj, lane)) & _M32
    x = x ^ (x >> 15)
    x = (x * _MUL1) & _M32  # int64 wrap-around keeps the low 32 bits exact
    x = x ^ (x >> 13)
    x = (x * _MUL2) & _M32
    x = x ^ (x >> 16)
    x = (x * _MUL3) & _M32
    x = x ^ (x >> 14)
    return x


def bits32_scalar(seed: int, obj: int, idx: int, lane: int = 0) -> int:
    """The same hash for one index, in plain Python integers."""
    x = (idx + _key(seed, obj, lane)) & _M32
    x ^= x >> 15
    x = (x * _MUL1) & _M32
    x ^= x >> 13
    x = (x * _MUL2) & _M32
    x ^= x >> 16
    x = (x * _MUL3) & _M32
    x ^= x >> 14
    return x


# --------------------------------------------------------------------------- values
def _normal_scale(sigma: float) -> np.float32:
    return np.float32(sigma / _IH4_STD)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns (finite inputs)."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))
    return (b >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f32(u16: np.ndarray) -> np.ndarray:
    return (u16.astype(np.uint32) << np.uint32(16)).view(np.float32)


def values_np(dist: tuple, seed: int, obj: int, start: int, count: int, dtype: str = "f32") -> np.ndarray:
    """Host spelling.  ``dist`` is ("uniform",) or ("normal", sigma).  Returns float32, or uint16
    bf16 bit patterns when ``dtype == "bf16"``."""
    if dist[0] == "uniform":
        u = (_bits32_np(seed, obj, start, count, 0) >> np.uint64(8)).astype(np.int64)
        v = (u - (1 << 23)).astype(np.float32) / np.float32(1 << 23)
    elif dist[0] == "normal":
        x0 = _bits32_np(seed, obj, start, count, 0)
        x1 = _bits32_np(seed, obj, start, count, 1)
        s = (x0 & np.uint64(0xFFFF)) + (x0 >> np.uint64(16)) + (x1 & np.uint64(0xFFFF)) + (x1 >> np.uint64(16))
        v = (s.astype(np.int64) - _IH4_MEAN).astype(np.float32) * _normal_scale(dist[1])
    elif dist[0] == "smallint":  # integer-valued fp32 in [-dist[1], dist[1]]: every summation order is exact
        r = int(dist[1])
        u = (_bits32_np(seed, obj, start, count, 0) >> np.uint64(8)).astype(np.int64)
        v = ((u % (2 * r + 1)) - r).astype(np.float32)
    else:
        raise ValueError(dist)
    if dtype == "bf16":
        return f32_to_bf16_bits(v)
    if dtype != "f32":
        raise ValueError(dtype)
    return v


def values_torch(dist: tuple, seed: int, obj: int, start: int, count: int, dtype: str = "f32",
                 device="cuda", out=None, slab: int = 1 << 24):
    """Device spelling of :func:`values_np` (torch integer ops; generated in slabs to bound scratch)."""
    import torch

    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    if out is None:
        out = torch.empty(count, dtype=tdt, device=device)
    for s0 in range(0, count, slab):
        n = min(slab, count - s0)
        if dist[0] == "uniform":
            u = _bits32_torch(seed, obj, start + s0, n, 0, device) >> 8
            v = (u - (1 << 23)).to(torch.float32) / float(1 << 23)
        elif dist[0] == "normal":
            x0 = _bits32_torch(seed, obj, start + s0, n, 0, device)
            x1 = _bits32_torch(seed, obj, start + s0, n, 1, device)
            s = (x0 & 0xFFFF) + (x0 >> 16) + (x1 & 0xFFFF) + (x1 >> 16)
            scale = torch.tensor(float(_normal_scale(dist[1])), dtype=torch.float32, device=device)
            v = (s - _IH4_MEAN).to(torch.float32) * scale
        elif dist[0] == "smallint":
            r = int(dist[1])
            u = _bits32_torch(seed, obj, start + s0, n, 0, device) >> 8
            v = ((u % (2 * r + 1)) - r).to(torch.float32)
        else:
            raise ValueError(dist)
        out[s0:s0 + n] = v.to(tdt)
    return out


# --------------------------------------------------------------------------- timelines
def uniform_offsets_ns(seed: int, n: int, window_ns: int = 1_000_000) -> list[int]:
    """n join offsets, uniform on [0, window_ns), integer nanoseconds."""
    return [bits32_scalar(seed, 0x4A01, i) * window_ns >> 32 for i in range(n)]


def exponential_arrivals_ns(seed: int, n: int, mean_ns: int = 5_000_000) -> list[int]:
    """n i.i.d. arrival times, exponential with the given mean, measured from the round start."""
    out = []
    for i in range(n):
        u = (bits32_scalar(seed, 0x4A02, i) + 0.5) / 4294967296.0
        out.append(int(round(-mean_ns * math.log1p(-u))))
    return out


# event kinds, in the order in which events with equal time are applied
EV_FAIL, EV_CREATE, EV_PUT, EV_REDUCE, EV_BROADCAST, EV_JOIN, EV_PROGRESS = range(7)


def sort_events(events: list[tuple]) -> list[tuple]:
    """Events are tuples ``(t_ns, kind, id, ...)``; equal times are ordered by kind, then id
    (failures first, then publications, then requests)."""
    return sorted(events, key=lambda e: (e[0], e[1], e[2]))


# --------------------------------------------------------------------------- the five workloads
@dataclass
class Workload:
    name: str
    kind: str                 # "reduce" | "broadcast" | "round" | "ft_reduce"
    dtype: str                # "f32" | "bf16"
    dist: tuple
    elems: int                # elements per object
    chunk_bytes: int
    degree: int
    n_objects: int = 0        # reduce sources
    k: int = 0                # objects reduced
    n_receivers: int = 0
    rounds: int = 1
    seed: int = BASE_SEED
    extra: dict = field(default_factory=dict)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def object_bytes(self) -> int:
        return self.elems * self.elem_bytes


def workload(name: str, **over) -> Workload:
    """The synthetic stand-ins for the five configurations (sizes and shapes only)."""
    if name == "cfg1":   # reduce microbenchmark shape at 1 MB
        w = Workload("cfg1", "reduce", "f32", ("uniform",), 262_144, 64 * KiB, 2, n_objects=8, k=8)
    elif name == "cfg2":  # broadcast microbenchmark + staggered joins
        w = Workload("cfg2", "broadcast", "f32", ("uniform",), 16_777_216, 1 * MiB, 2, n_receivers=16,
                     extra={"join_window_ns": 1_000_000})
    elif name == "cfg3":  # async-SGD: first half of the workers, ResNet-50-sized gradient
        w = Workload("cfg3", "reduce", "f32", ("normal", 1e-3), 25_557_032, 4 * MiB, 2, n_objects=16, k=8,
                     rounds=50, extra={"mean_arrival_ns": 5_000_000})
    elif name == "cfg4":  # RL policy round: broadcast then reduce, bf16
        w = Workload("cfg4", "round", "bf16", ("normal", 0.02), 33_554_432, 2 * MiB, 4, n_objects=64, k=64,
                     n_receivers=64)
    elif name == "cfg5":  # fault-tolerant reduce; elems set per size by the caller
        w = Workload("cfg5", "ft_reduce", "f32", ("uniform",), 256, 4 * MiB, 2, n_objects=32, k=32,
                     extra={"fail_worker": 7, "fail_fraction": 0.4,
                            "sizes_bytes": [KiB * 4 ** j for j in range(11)]})
    else:
        raise KeyError(name)
    for key, val in over.items():
        setattr(w, key, val)
    return w


def cfg5_at(size_bytes: int) -> Workload:
    w = workload("cfg5")
    w.elems = size_bytes // 4
    w.chunk_bytes = min(4 * MiB, size_bytes)
    return w


def n_chunks(nbytes: int, chunk_bytes: int) -> int:
    return (nbytes + chunk_bytes - 1) // chunk_bytes
