"""Host-side logic of the multi-rank benchmark path on CPU (gloo, world size 2): the timing reduction takes
the maximum over ranks, and the reference arm runs on rank 0 only."""
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    got = bench.max_over_ranks([10.0 + rank, 5.0 - rank], "cpu")
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, got))


def test_max_over_ranks_gloo_world_size_2():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29611, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0] == results[1] == [11.0, 5.0]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg0",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_plain_start_with_several_gpus_becomes_a_launcher():
    """`python bench.py --gpus N` without torchrun's environment starts N ranks of itself (one process per GPU)."""
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.spawn_command(["--gpus", "4", "--steps", "2"], 4, 29999)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "4", "--steps", "2"]
    assert cmd[cmd.index("--master-port") + 2].endswith("bench.py")
    # under torchrun (WORLD_SIZE set) the script must NOT spawn again: the reference arm on rank 1 simply returns
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                        "--workload", "cfg0", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_block_count_fills_about_two_seconds():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.plan_blocks(20, 18.0) == 7          # 0.36 s blocks: 6 needed, made odd
    assert bench.plan_blocks(20, 200.0) == 1         # a 4 s block is enough
    assert bench.plan_blocks(20, 0.9) == 9           # capped
