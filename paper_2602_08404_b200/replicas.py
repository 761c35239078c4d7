"""Multi-GPU bookkeeping of the measurement: the path runs as independent replicas, one process per GPU.

Sequences are independent, so N GPUs run N copies of the workload with no exchange on the data path; the
only collective work is the barrier around the timed region and the maximum of the per-rank times.  These
helpers hold that logic so that it can be exercised on CPU with the gloo backend.
"""
import torch
import torch.distributed as dist


def world_size():
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def max_over_ranks(value, device="cpu"):
    """The slowest rank's value (a time): what a whole-job rate has to be computed from."""
    if world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step, ms_per_step):
    """Units per second over all replicas, from the slowest rank's time per step (weak scaling)."""
    return world_size() * units_per_rank_per_step / (ms_per_step * 1e-3)


def barrier():
    if world_size() > 1:
        dist.barrier()


def launcher_command(script, argv, n, port=None, python=None):
    """The command that runs `script argv...` as n ranks of one node (one process per GPU), rendezvous on
    127.0.0.1: what `--gpus n` means when no launcher has set WORLD_SIZE yet."""
    import os
    import sys
    port = port or 29500 + os.getpid() % 20000
    return [python or sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n)}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), script] + list(argv)


def needs_launcher(n_requested, env=None):
    """True when more than one replica was asked for and this process was not started by a launcher."""
    import os
    env = os.environ if env is None else env
    return int(n_requested) > 1 and "WORLD_SIZE" not in env


def run_under_launcher(script, argv, n, timeout=None, port=None):
    """Runs the script as n ranks and passes its output through; returns the launcher's exit code."""
    import subprocess
    return subprocess.run(launcher_command(script, argv, n, port=port), timeout=timeout).returncode
