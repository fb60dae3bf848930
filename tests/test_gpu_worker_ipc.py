"""Worker-per-GPU mode with real CUDA IPC mappings: two PROCESSES, both on the one GPU there is, map each other's arena
and objects (hpl_ipc_export / hpl_ipc_import), replicate the timeline and run their own tasks level by level with a
barrier between levels (gloo).  No kernel waits for another process.  Values are checked against the oracle in every
process; the bench's own worker-per-GPU round is run the same way."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import numpy as np
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    import bench
    import paper_2002_05814_b200 as hpl
    from oracle.store import OracleStore, DT_F32
    from tests.harness import gen

    elems, chunk, k, R = 7 * 4096 + 9, 16 << 10, 4, 2
    arena_bytes = 32 << 20
    arena = torch.empty(arena_bytes, dtype=torch.uint8, device="cuda")
    host = {i: gen(("uniform",), 500, i, elems) for i in range(k)}
    mine = {i: torch.from_numpy(host[i]).cuda() for i in range(k) if i % world == rank}          # worker i lives on rank i % world
    recv = {j: torch.zeros(elems, dtype=torch.float32, device="cuda") for j in range(R) if j % world == rank}
    torch.cuda.synchronize()
    exported = {"arena": hpl.ipc_export(arena.data_ptr()), "obj": {i: hpl.ipc_export(t.data_ptr()) for i, t in mine.items()},
                "recv": {j: hpl.ipc_export(t.data_ptr()) for j, t in recv.items()}}
    everyone = [None] * world
    dist.all_gather_object(everyone, exported)
    addr_obj, addr_recv, mapped = {}, {}, []
    c = hpl.Context(chunk, 2, 2, arena=arena.data_ptr(), arena_bytes=arena_bytes, stream=torch.cuda.current_stream().cuda_stream,
                    fuse=False, rank=rank, world_size=world)
    for r in range(world):
        if r == rank:
            addr_obj.update({i: t.data_ptr() for i, t in mine.items()})
            addr_recv.update({j: t.data_ptr() for j, t in recv.items()})
            continue
        p = hpl.ipc_import(*everyone[r]["arena"])
        mapped.append(p)
        c.set_peer_arena(r, p)
        for i, h in everyone[r]["obj"].items():
            addr_obj[i] = hpl.ipc_import(*h)
            mapped.append(addr_obj[i])
        for j, h in everyone[r]["recv"].items():
            addr_recv[j] = hpl.ipc_import(*h)
            mapped.append(addr_recv[j])
    o = OracleStore(chunk, 2, 2)
    for i in range(k):
        c.create(i, i, elems * 4)
        o.create(i, i, elems * 4, DT_F32)
    for j in range(R):
        c.create(50 + j, j, elems * 4)
        o.create(50 + j, j, elems * 4, DT_F32)
    c.reduce(100, list(range(k)), k)
    o.reduce(100, list(range(k)), k)
    c.broadcast(100, [50 + j for j in range(R)])
    o.broadcast(100, [50 + j for j in range(R)])
    for j in range(R):
        c.join(50 + j, addr_recv[j])
        o.join(50 + j)
    for i in range(k):
        c.advance(i + 1)
        o.advance(i + 1)
        c.put(i, addr_obj[i], elems * 4)
        o.put(i, host[i], elems * 4)
    c.drive(dist.barrier)
    want = o.get(100)
    ptr, n = c.get(100)
    if 100 % world == rank:                                     # the output lives here: read it
        off = ptr - arena.data_ptr()
        got = arena[off:off + n].cpu().numpy().view(np.uint32)
        assert np.array_equal(got, want.view(np.uint32)), "reduce across processes differs from the oracle"
    for j, t in recv.items():                                   # my receivers, written by whoever ran the root task
        c.get(50 + j)
        assert t.cpu().numpy().tobytes() == want.tobytes(), "receiver differs"
    assert c.schedule_dump(100) == o.dump(100)
    st = c.stats()
    total = torch.tensor([st["reduce_tasks"]], dtype=torch.int64)
    dist.all_reduce(total)
    assert int(total) == 2                                       # the tree of 4 has two internal nodes: each was run once, by its owner
    c.shutdown()
    dist.barrier()
    for p in mapped:
        hpl.ipc_close(p)
    dist.barrier()
    # the bench's own round, same plumbing (gloo stands in for NCCL: both ranks share the GPU)
    out = bench.worker_per_gpu_round(dist, torch.device("cuda", 0), rank, world, steps=2, object_bytes=4 << 20)
    assert "error" not in out and out["ms_per_reduce"] > 0, out
    with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
        f.write("ok")
    dist.destroy_process_group()


def test_two_processes_on_one_gpu_map_each_others_memory(tmp_path):
    from paper_2002_05814_b200 import build
    build.build()
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok0").exists() and (tmp_path / "ok1").exists()
