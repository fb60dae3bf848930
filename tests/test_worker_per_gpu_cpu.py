"""Worker-per-GPU mode on CPU (gloo, schedule-only contexts): every rank applies the same timeline, plans the same
levels and releases only the tasks whose output (reduce) or source copy (fan-out) it owns.  Checked: the ranks' tasks
together are exactly the plan of a single context, nobody's share overlaps, schedules stay identical, and the
survivors finish after a rank has left between two plans."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHUNK, S = 4096, 5 * 4096 + 64


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _timeline(c, world, fail_rank_after=None, barrier=lambda: None, live=None):
    """8 workers (worker w on rank w % world), a Reduce of their objects whose output is broadcast to 4 receivers."""
    import paper_2002_05814_b200 as hpl
    k, R = 8, 4
    for i in range(k):
        c.create(i, i, S)
    for j in range(R):
        c.create(50 + j, 20 + j, S)
    c.reduce(100, list(range(k)), k)
    c.broadcast(100, [50 + j for j in range(R)])
    for i in range(k):
        c.advance(i + 1)
        c.put(i, 4096 * (i + 1), S if i != 5 else 2 * CHUNK)        # object 5 is only partly there
    for j in range(R):
        c.advance(20 + j)
        c.join(50 + j, 1 << 30)
    c.drive(barrier)
    if fail_rank_after is not None:
        c.fail_rank(fail_rank_after)
    c.advance(100)
    if hpl.HPL_OK == 0 and (fail_rank_after is None or 5 % world != fail_rank_after):
        c.put(5, 4096 * 6, S)
    c.drive(barrier)


def _worker(rank, world, port, out_dir, leaver):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_2002_05814_b200 as hpl

    survivors = dist.new_group([r for r in range(world) if r != leaver]) if leaver is not None else None
    # the plan of a single context (world 1), for reference, with every node's result materialised (the paper's shape)
    ref = hpl.Context(CHUNK, 2, 2, fuse=False)
    _timeline(ref, 1)
    ref_stats = ref.stats()
    ref_dump = ref.schedule_dump(100)
    ref.shutdown()

    c = hpl.Context(CHUNK, 2, 2, fuse=False, rank=rank, world_size=world)
    phase = {"n": 0}

    def barrier():
        dist.barrier(group=survivors if (phase["n"] and survivors is not None) else None)

    if leaver is None:
        _timeline(c, world, None, barrier)
    else:
        # first part with everyone; then `leaver` goes away between two plans and the others take it out
        k, R = 8, 4
        for i in range(k):
            c.create(i, i, S)
        for j in range(R):
            c.create(50 + j, 20 + j, S)
        c.reduce(100, list(range(k)), k)
        c.broadcast(100, [50 + j for j in range(R)])
        for i in range(k):
            c.advance(i + 1)
            c.put(i, 4096 * (i + 1), S if i != 5 else 2 * CHUNK)
        for j in range(R):
            c.advance(20 + j)
            c.join(50 + j, 1 << 30)
        c.drive(barrier)
        dist.barrier()
        if rank == leaver:
            c.shutdown()
            with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
                f.write("left")
            dist.destroy_process_group()
            return
        phase["n"] = 1
        c.advance(100)
        c.fail_rank(leaver)
        if 5 % world != leaver:
            c.put(5, 4096 * 6, S)
        c.drive(barrier)
    group = survivors if leaver is not None else None
    n_live = world - (1 if leaver is not None else 0)
    st = c.stats()
    mine = torch.tensor([st["reduce_tasks"], st["fanout_tasks"], st["bytes_read_planned"], st["bytes_written_planned"]], dtype=torch.int64)
    total = mine.clone()
    dist.all_reduce(total, group=group)
    words = torch.tensor(c.schedule_dump(100), dtype=torch.int64)
    gathered = [torch.zeros_like(words) for _ in range(n_live)]
    dist.all_gather(gathered, words, group=group)
    assert all(torch.equal(g, words) for g in gathered), "schedules differ between ranks"
    rc, _, _ = c.try_get(100)
    if leaver is None:
        # together the ranks did exactly what one context does alone, and every rank did something
        assert total.tolist() == [ref_stats["reduce_tasks"], ref_stats["fanout_tasks"], ref_stats["bytes_read_planned"],
                                  ref_stats["bytes_written_planned"]], (total.tolist(), ref_stats)
        assert list(words) == ref_dump
        most = mine.clone()
        dist.all_reduce(most, op=dist.ReduceOp.MAX, group=group)
        assert most[0] < total[0]                      # the tree's nodes are spread over the ranks
        assert rc == hpl.HPL_ERR_CUDA                  # complete: only the device is missing
        for j in range(4):
            assert c.try_get(50 + j)[0] == hpl.HPL_ERR_CUDA
    else:
        # the output lives on rank 100 % world: lost with it, else the survivors' sum is complete
        assert rc == (hpl.HPL_ERR_FAILED_WORKER if 100 % world == leaver else hpl.HPL_ERR_CUDA), rc
    c.shutdown()
    dist.barrier(group=group)
    with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
        f.write("ok")
    dist.destroy_process_group()


def _run(world, tmp_path, leaver=None):
    from paper_2002_05814_b200 import build
    build.build()
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path), leaver), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))


def test_two_ranks_share_the_plan(tmp_path):
    _run(2, tmp_path)


def test_four_ranks_share_the_plan(tmp_path):
    _run(4, tmp_path)


def test_a_rank_leaves_between_plans_and_the_survivors_finish(tmp_path):
    _run(4, tmp_path, leaver=3)


def test_the_rank_that_holds_the_output_leaves(tmp_path):
    _run(4, tmp_path, leaver=0)
