"""The N > 1 benchmark path on CPU: the path is "replicas only", so all the ranks share is a
barrier and the max-over-ranks of their measured time.  Two gloo ranks exercise exactly that
code (bench.RankSync), and the reference arm's non-zero ranks must exit silently."""
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    sync = bench.RankSync(dist, "cpu")
    sync.barrier()
    local_ms = 40.0 + 5.0 * rank                 # the slower replica sets the job's step time
    ms = sync.max(local_ms)
    value = bench.whole_job_tokens_per_s(8 * 1024, world, ms)
    sync.barrier()
    out.put((rank, ms, value))
    dist.destroy_process_group()


def test_two_gloo_ranks_share_max_time_and_sum_tokens():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in results:
        assert ms == 45.0                                        # max over ranks, on every rank
        assert abs(value - 2 * 8192 / 0.045) < 1e-6              # whole-job tokens/s: both replicas' tokens
    import bench
    assert bench.RankSync(None, "cpu").max(3.25) == 3.25         # single rank: identity, no process group


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
