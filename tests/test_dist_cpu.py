"""World-size-2 gloo test of the benchmark's process-group plumbing (runs on CPU)."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2605_08565_b200 import dist
    r, lr, w = dist.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    dist.barrier()
    # rank r processed (r+1)*1000 units in (r+1)*0.5 s: whole job = 3000 units / max time 1.0 s
    value, t = dist.whole_job_throughput((rank + 1) * 1000.0, (rank + 1) * 0.5)
    import torch
    amax = dist.global_amax(torch.tensor([1.5 + rank], dtype=torch.float32))
    mse = dist.global_mse(10.0 * (rank + 1), 60)
    assert float(amax) == 2.5 and mse == 0.5, (float(amax), mse)
    out.put((rank, value, t, dist.reduce_max(rank), dist.reduce_sum(rank + 1)))
    dist.barrier()
    dist.shutdown()


def test_two_rank_reductions_over_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, t, mx, sm in res:
        assert value == 3000.0 and t == 1.0 and mx == 1.0 and sm == 3.0


def test_rank_seeds_never_collide_and_single_process_is_a_no_op():
    from paper_2605_08565_b200 import dist
    seeds = {dist.rank_seed(2, r, i) for r in range(8) for i in range(8)}
    assert len(seeds) == 64
    assert dist.reduce_max(3.5) == 3.5 and dist.reduce_sum(2.0) == 2.0
    assert dist.whole_job_throughput(10.0, 2.0) == (5.0, 2.0)
    # row shards tile the rows without gaps or overlap
    for rows, world in ((4096, 8), (1000, 3), (7, 8)):
        edges = [dist.row_shard(rows, r, world) for r in range(world)]
        assert edges[0][0] == 0 and edges[-1][1] == rows
        assert all(a[1] == b[0] for a, b in zip(edges[:-1], edges[1:]))
    assert dist.global_mse(12.0, 48) == 0.25


def test_bench_starts_its_own_ranks_when_not_under_torchrun(tmp_path):
    """`bench.py --gpus N` outside a torchrun environment re-launches itself as N ranks; checked here with
    a stand-in script that records the environment every rank was given."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "rank_probe.py"
    script.write_text(
        "import os, sys\n"
        "open(os.path.join(sys.argv[1], 'rank' + os.environ['RANK']), 'w').write("
        "' '.join([os.environ['WORLD_SIZE'], os.environ['LOCAL_RANK'], os.environ['MASTER_ADDR'], sys.argv[2]]))\n")
    code = ("import sys; sys.path.insert(0, %r); import bench; "
            "sys.exit(bench.spawn_ranks(2, %r, [%r, '--steps=7']))" % (root, str(script), str(tmp_path)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    assert subprocess.run([sys.executable, "-c", code], env=env, timeout=300).returncode == 0
    for r in range(2):
        assert (tmp_path / f"rank{r}").read_text() == f"2 {r} 127.0.0.1 --steps=7"
