#!/usr/bin/env python
"""Benchmark of the TEAM MoE-layer step on B200.

Workload: the SDAR-30B-A3B-shaped MoE layer (hidden 2048, 128 experts top-8, SwiGLU intermediate 768,
bf16 weights, fp32 router), batch 1, block of 4 tokens, the scripted 4-step denoising schedule (one
token accepted per step), TEAM's activation rule on (delayed caching + limited activation).  One
"step" is one pass of the whole hot path -- router, selection/dispatch, grouped SwiGLU experts,
weighted combine -- i.e. one call of team_moe_forward for one denoising step of one layer.  Successive
steps cycle through the 4 denoising steps and through R independent layers (R sets of weights,
~1.2 GB each) so that expert weights always come from HBM, never from L2.

Prints ONE JSON line (rank 0).  `value` = rows presented per second over all GPUs, inputs resident in
HBM; `e2e` = the same through the C ABI with host buffers (pinned host -> device copies of the step's
inputs and a device -> host read of y inside the timed region); `roofline` = the expert kernel's
achieved HBM bandwidth on activated-expert weight bytes; `cpu_baseline` = the oracle on host cores.
`--impl reference` times the oracle instead (it is the reference arm for this build).
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "MoE-layer tokens/s per denoising step (rows presented / s)"
UNIT = "tokens/s"
WORKLOAD = "c2_sdar_bf16: H2048 E128 top8 I768 bf16, batch 1 x block 4, 4 denoising steps, TEAM (DCD|LAC)"
TEAM_FLAGS = 3


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8000)
    ap.add_argument("--warmup", type=int, default=400)
    ap.add_argument("--impl", default="team", choices=["team", "reference"])
    ap.add_argument("--layers", type=int, default=8, help="independent weight sets cycled through (L2 defeat)")
    ap.add_argument("--flags", type=int, default=TEAM_FLAGS, help="0 vanilla, 1 DCD, 3 DCD|LAC")
    ap.add_argument("--no-graph", action="store_true", help="issue every step as separate calls (no CUDA graph)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="budget of the oracle baseline leg")
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c4", "paper"],
                    help="c2: the headline step (default); c3: 256 experts + shared, block 32; c4: c2 shape, --seqs x 4 branches x 4; paper: c2 shape, block 32 x 4 branches in one group")
    ap.add_argument("--seqs", type=int, default=1, help="sequences of the c4 batch sweep")
    return ap.parse_args()


def sm_max_hz():
    """Maximum SM clock in Hz (for sizing the device-side delay); 1.965 GHz if NVML is not there."""
    try:
        import pynvml
        pynvml.nvmlInit()
        h = pynvml.nvmlDeviceGetHandleByIndex(int(os.environ.get("LOCAL_RANK", "0")))
        return pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM) * 1e6
    except Exception:
        return 1.965e9


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed regions run."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                 "sw_thermal_slowdown": 0x20, "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                util = nv.nvmlDeviceGetUtilizationRates(self.h).gpu
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((mhz, util))
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(0.02)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        busy = [m for m, u in self.samples if u > 0] or [m for m, _ in self.samples]
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_leg(args, shape, weights_host, steps, budget_s):
    """Times the oracle, as it stands, on the host cores over a bounded sample of the same workload."""
    from oracle import team_oracle as O
    from tests import _parity as P
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = len(os.sched_getaffinity(0))
    ocfg = P.oracle_config(shape, args.flags)
    t_total, n = 0.0, 0
    y_prev = None
    while t_total < budget_s and n < 400:
        step = steps[n % len(steps)]
        t0 = time.perf_counter()
        y_prev, _ = O.moe_forward(ocfg, weights_host, step["x"], step["tok_state"], step["conf"], step["pos"],
                                  step["group"], step["branch"], y_prev=y_prev if n % len(steps) else None)
        t_total += time.perf_counter() - t0
        n += 1
    rows = shape.rows
    return {"value": rows * n / t_total, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} layer-steps of the same schedule on one layer's weights ({t_total:.1f} s of CPU time)"}, \
        t_total / n


def run_reference(args):
    """The reference arm: the CPU oracle on the bench workload (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2602_08404_b200 import workloads as W
    shape = W.C2
    weights = W.make_weights(shape)
    steps = W.make_schedule(shape)
    budget = max(5.0, min(120.0, 0.05 * (args.steps + args.warmup)))
    cb, s_per_step = oracle_leg(args, shape, weights, steps, budget)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": 0,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": s_per_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD, "flags": args.flags},
            "cpu_baseline": cb,
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2602_08404_b200 import binding as B
    from paper_2602_08404_b200 import replicas as R_
    from paper_2602_08404_b200 import build as build_mod
    from paper_2602_08404_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the TEAM library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build_mod.build()
    if world > 1:
        dist.barrier()
    dev = torch.device("cuda", local_rank)

    shape = {"c2": W.C2, "c3": W.C3, "c4": W.c4(args.seqs), "paper": W.paper_point()}[args.workload]
    T, H, E, k, I = shape.rows, shape.hidden, shape.n_experts, shape.top_k, shape.inter
    ns = shape.n_shared
    workload = WORKLOAD if args.workload == "c2" else (
        f"{shape.name}: H{H} E{E}{'+%d shared' % ns if ns else ''} top{k} I{I} bf16, {shape.seqs} seq x {shape.branches} "
        f"branches x block {shape.block} = {T} rows, {shape.n_steps} denoising steps, flags {args.flags}")
    steps_host = W.make_schedule(shape)                      # the scripted denoising steps, seeded
    n_sched = len(steps_host)
    R = args.layers

    # R independent layers, generated on the device (seeded); layer 0 also goes to the host for the oracle leg
    gen = torch.Generator(device=dev)
    layers, packed = [], []
    for r in range(R):
        gen.manual_seed(1000 + r)
        wr = (torch.randn((E, H), generator=gen, device=dev, dtype=torch.float32) * 0.02).contiguous()
        wg, wu, wd = [(torch.randn(s, generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)
                      for s in ((E + ns, I, H), (E + ns, I, H), (E + ns, H, I))]
        layers.append((wr, wg, wu, wd if r == 0 else None))
        packed.append(B.team_pack_w_down(wd))      # the layout the library reads; row-major kept for the oracle leg
    cfg = B.make_config(H, E, k, I, ns, max_rows=T, max_groups=shape.seqs, dtype=B.TEAM_DTYPE_BF16, flags=args.flags,
                        tau_hot=shape.tau_hot, L_hot=shape.L_hot)
    ctxs = []
    for r in range(R):
        c = B.team_create(cfg)
        B.team_set_weights(c, *layers[r][:3], packed[r])
        ctxs.append(c)

    x_dev = [B.to_device(s["x"], B.TEAM_DTYPE_BF16, dev) for s in steps_host]
    st_dev = [B.state_to_device(s, dev) for s in steps_host]
    y_dev = torch.zeros((T, H), dtype=torch.float32, device=dev)

    # the cycle: combo i = (layer i % R, denoising step i % n_sched), period lcm(R, n_sched)
    period = int(np.lcm(R, n_sched))
    combos = [(i % R, i % n_sched) for i in range(period)]

    def one_step(i, out=None):
        r, s = combos[i % period]
        B.team_moe_forward(ctxs[r], x_dev[s], st_dev[s], out, y_dev)

    # activated experts per combo (deterministic), for the bytes accounting
    n_act, n_rows = [], []
    for i in range(period):
        out = B.alloc_routing(cfg, T, dev)
        one_step(i, out)
        torch.cuda.synchronize()
        n_act.append(int(out["n_active"].item()))
        n_rows.append(int(out["n_rows_active"].item()))
        code, detail = B.team_read_status(ctxs[combos[i][0]])
        if code != 0:
            raise SystemExit(f"device status {code} detail {detail}")
    one_step(0)                                   # as the timed steps run: no exports
    torch.cuda.synchronize()
    launches_per_step = B.team_last_launch_count(ctxs[0])
    bytes_per_expert = 3 * H * I * 2

    # CUDA graph of one full cycle (period steps); replayed for the timed region
    graph = None
    if not args.no_graph:
        try:
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for i in range(period):
                    one_step(i)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(period):
                    one_step(i)
            graph = g
        except Exception as e:                                   # report, and time plain launches instead
            print(f"[bench] CUDA graph capture failed ({e}); timing plain launches", file=sys.stderr)
            graph = None

    def run_steps(n):
        """Issues exactly n steps: whole cycles as graph replays, the remainder as plain calls."""
        if graph is None:
            for i in range(n):
                one_step(i)
            return n
        for _ in range(n // period):
            graph.replay()
        for i in range(n % period):
            one_step(i)
        return n

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    with sampler:
        # ---- device-resident timing -----------------------------------------------------------------
        run_steps(max(args.warmup, 3))
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        issued = run_steps(args.steps)
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1)
        ms_per_step = ms / issued
        ms_per_step = R_.max_over_ranks(ms_per_step, dev)

        # ---- expert-kernel duration (CUDA events around every launch, on the launching stream) -------
        for c in ctxs:
            B.team_expert_timing(c, 1)
        # These steps are plain launches with event records in between: about five stream operations per step.
        # A host slower than the GPU would leave the GPU waiting between the first event and the kernel, and that
        # wait would be counted as kernel time.  So the stream is held back for a moment (a bounded device-side
        # spin) while the host queues the whole batch, and the batch is kept below the launch queue's depth.
        n_roof = min(args.steps, 18 * period)
        n_roof -= n_roof % period
        n_roof = max(n_roof, period)
        torch.cuda.synchronize()
        torch.cuda._sleep(int(sm_max_hz() * 0.012))            # ~12 ms; the host needs a few ms for the batch
        for i in range(n_roof):
            one_step(i)
        tot_ms, tot_n = 0.0, 0
        for c in ctxs:
            avg, n = B.team_expert_timing(c, 0)
            tot_ms += avg * n
            tot_n += n
        kernel_ms = tot_ms / max(tot_n, 1)

        # ---- end to end through the C ABI with host buffers -------------------------------------------
        x_pin = [torch.as_tensor(s["x"]).to(torch.bfloat16).pin_memory() for s in steps_host]
        st_pin = [{n: torch.as_tensor(np.ascontiguousarray(v)).pin_memory() for n, v in
                   (("tok_state", s["tok_state"].astype(np.uint8)), ("conf", s["conf"].astype(np.float32)),
                    ("pos", s["pos"].astype(np.int32)), ("group", s["group"].astype(np.int32)),
                    ("branch", s["branch"].astype(np.int32)))} for s in steps_host]
        y_pin = torch.zeros((T, H), dtype=torch.float32).pin_memory()
        # bytes the library moves per step: its staging block pads x and each state array to 256 bytes
        pad = lambda n: (n + 255) // 256 * 256
        h2d = pad(x_pin[0].numel() * 2) + sum(pad(v.numel() * v.element_size()) for v in st_pin[0].values())
        d2h = y_pin.numel() * 4

        def e2e_step(i):
            r, s = combos[i % period]
            # host buffers in, host buffer out: the library stages, copies, runs the layer, copies back and synchronises
            B.team_moe_forward_host(ctxs[r], x_pin[s], st_pin[s], None, y_pin)

        n_e2e = max(period, min(args.steps, 2000))
        # on a stream of its own: the library records the step (copy in, kernels, copy out) as a graph, which the
        # legacy default stream cannot do
        e2e_stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(e2e_stream):
            for i in range(max(3, min(args.warmup, 100))):
                e2e_step(i)
            barrier()
            t0 = time.perf_counter()
            for i in range(n_e2e):
                e2e_step(i)
            barrier()
            e2e_ms_per_step = (time.perf_counter() - t0) * 1e3 / n_e2e
        e2e_ms_per_step = R_.max_over_ranks(e2e_ms_per_step, dev)
    clocks = sampler.summary()

    # ---- accounting ------------------------------------------------------------------------------
    mean_act = float(np.mean(n_act))
    mean_rows = float(np.mean(n_rows))
    algo_bytes = mean_act * bytes_per_expert                      # activated-expert weight bytes per launch
    peak, peak_kind = measured_peaks()
    achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
    value = R_.whole_job_rate(T, ms_per_step)
    stream_kernel = H in (1024, 2048)      # the library's choice: weight-streaming kernel (resident or gather mode)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload, "flags": args.flags, "rows_presented": T, "rows_computed_mean": mean_rows,
                   "activated_experts_mean": mean_act, "layers_cycled": R,
                   "l2": f"inputs larger than L2: weights rotate over {R} layers ({R * E * bytes_per_expert / 1e9:.1f} GB)",
                   "cuda_graph": graph is not None, "steps_issued": issued, "parallelism": f"replicas x{world}"},
        "clocks": clocks,
        "e2e": {"value": R_.whole_job_rate(T, e2e_ms_per_step), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms_per_step, "steps": n_e2e},
        "gpu_launches": launches_per_step * issued,
        "activated_experts_per_s": R_.whole_job_rate(mean_act, ms_per_step),
        "rows_computed_per_s": R_.whole_job_rate(mean_rows, ms_per_step),
        "step_hbm_frac": (algo_bytes + 4 * E * H) / (ms_per_step * 1e-3) / 1e9 / peak,
        "roofline": {"bound": "hbm", "kernel": "k_experts_stream" if stream_kernel else "k_experts_tc", "achieved": achieved, "peak": peak,
                     "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_8TBs_nominal": achieved / 8000.0, "kernel_ms": kernel_ms,
                     "algorithmic_bytes_per_launch": algo_bytes, "launches_timed": tot_n,
                     # DRAM read + write bytes per launch: ncu capture at 16 activated experts (151.08 MB read +
                     # 3.25 MB written, profiles/experts_stream_c2_bench.md), scaled to this run's mean
                     "traffic": mean_act * (151.08e6 + 3.25e6) / 16.0 if args.workload == "c2" else None,
                     # the same launches as a contraction: 6 H I flops per token-slot (routed and shared)
                     "tensor_tflops": mean_rows * (k + ns) * 6.0 * H * I / (kernel_ms * 1e-3) / 1e12},
    }

    if rank == 0:
        if world == 1 and args.cpu_seconds > 0:
            weights_host = {n: t.float().cpu().numpy() for n, t in
                            zip(("w_router", "w_gate", "w_up", "w_down"), layers[0])}
            cb, _ = oracle_leg(args, shape, weights_host, steps_host, args.cpu_seconds)
            line["cpu_baseline"] = cb
        print(json.dumps(line))
    for c in ctxs:
        B.team_destroy(c)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
