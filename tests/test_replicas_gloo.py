"""The N > 1 path of the measurement on CPU: two gloo ranks, no GPU.

The hot path does not shard: N GPUs run N independent replicas, and the only collective work is the
barrier and the maximum over the ranks' times.  The test runs that bookkeeping with world_size 2 and
checks the whole-job rate against the definition (units of all ranks / slowest rank's time); it also
checks that the reference arm stays silent on ranks other than 0.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2602_08404_b200 import replicas as R
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        R.barrier()
        local_ms = 0.040 + 0.010 * rank              # rank 1 is the slow one
        ms = R.max_over_ranks(local_ms)
        rate = R.whole_job_rate(4, ms)               # 4 rows per rank and step
        out.put((rank, R.world_size(), ms, rate))
        R.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_rate_is_all_units_over_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, ms, rate in got:
        assert world == 2
        assert abs(ms - 0.050) < 1e-12                            # the maximum, on every rank
        assert abs(rate - 2 * 4 / 0.050e-3) < 1e-6                # 8 rows per step over 50 us


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2602_08404_b200 import replicas as R
    assert R.world_size() == 1
    assert R.max_over_ranks(0.25) == 0.25
    assert R.whole_job_rate(4, 0.04) == 4 / 0.04e-3
    R.barrier()


def test_reference_arm_prints_nothing_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    assert r.stdout.strip() == ""


def test_gpus_flag_without_a_launcher_starts_the_replicas_itself():
    """`--gpus 2` with no WORLD_SIZE in the environment: the same arguments are re-run as 2 ranks under
    torch.distributed.run (rendezvous on 127.0.0.1) and rank 0 prints the one line."""
    sys.path.insert(0, ROOT)
    from paper_2602_08404_b200 import replicas as R
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    assert R.needs_launcher(2, env) and not R.needs_launcher(1, env)
    assert not R.needs_launcher(2, dict(env, WORLD_SIZE="2"))          # already under a launcher
    stub = os.path.join(ROOT, "tests", "_replica_stub.py")
    cmd = R.launcher_command(stub, ["--gpus", "2", "--steps", "7"], 2, port=29500 + (os.getpid() + 977) % 2000)
    assert "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                             # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["asked"] == 2 and lines[0]["steps"] == 7
    assert abs(lines[0]["ms_per_step"] - 0.050) < 1e-12
    assert abs(lines[0]["value"] - 2 * 4 / 0.050e-3) < 1e-6


def test_bench_hands_gpus_n_to_the_launcher(monkeypatch):
    """bench.py --gpus 2, started plainly: before touching any device it re-runs itself under the launcher with the
    same arguments and exits with the launcher's code."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_08404_b200 import replicas as R
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    seen = {}

    def fake(script, argv, n, **kw):
        seen.update(script=script, argv=list(argv), n=n)
        return 17

    monkeypatch.setattr(R, "run_under_launcher", fake)
    try:
        bench.main(["--gpus", "2", "--steps", "20", "--warmup", "5"])
        raise AssertionError("bench.main should have exited")
    except SystemExit as e:
        assert e.code == 17
    assert seen["n"] == 2 and seen["argv"] == ["--gpus", "2", "--steps", "20", "--warmup", "5"]
    assert os.path.basename(seen["script"]) == "bench.py"


def _ep_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2602_08404_b200 import ep as EP
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        T, H = 5, 8
        tok_class = torch.tensor([1, 0, 2, 1, 0], dtype=torch.uint8)           # rows 1 and 4 were not computed
        y = torch.full((T, H), 100.0 + rank)                                    # what the rank's y held before the step
        y[tok_class != 0] = torch.arange(T * H, dtype=torch.float32).view(T, H)[tok_class != 0] * (rank + 1)
        got = EP.combine_partial_outputs(y, tok_class)
        out.put((rank, got.numpy().copy(), EP.expert_range(128, rank, world)))
    finally:
        dist.destroy_process_group()


def test_expert_parallel_outputs_are_summed_on_the_computed_rows_only():
    """The exchange step of expert-parallel sharding (two gloo ranks on CPU): computed rows become the sum of the
    ranks' partial sums, rows that were not computed keep each rank's own previous values."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() + 313) % 2000
    procs = [ctx.Process(target=_ep_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((out.get(timeout=120) for _ in procs), key=lambda g: g[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    base = torch.arange(40, dtype=torch.float32).view(5, 8).numpy()
    for rank, y, rng in got:
        for t in (0, 2, 3):
            assert (y[t] == base[t] * 3).all()                   # 1x + 2x
        for t in (1, 4):
            assert (y[t] == 100.0 + rank).all()
        assert rng == (64 * rank, 64 * rank + 64)
