#!/usr/bin/env python
"""Benchmark of the TEAM MoE-layer step on B200.

Headline workload (the default): the SDAR-30B-A3B-shaped MoE layer (hidden 2048, 128 experts top-8, SwiGLU
intermediate 768, bf16 weights, fp32 router), batch 1, block of 4 tokens, the scripted 4-step denoising
schedule (one token accepted per step), TEAM's activation rule on (delayed caching + limited activation).
One "step" is one pass of the whole hot path -- router, selection/dispatch, grouped SwiGLU experts, weighted
combine -- i.e. one call of team_moe_forward for one denoising step of one layer.  Successive steps cycle
through the 4 denoising steps and through R independent layers (R sets of weights, ~1.2 GB each) so that expert
weights always come from HBM, never from L2.

Prints ONE JSON line (rank 0).  `value` = rows presented per second over all GPUs, inputs resident in HBM;
`e2e` = the same through the C ABI with host buffers (pinned host -> device copies of the step's inputs and a
device -> host read of y inside the timed region); `roofline` = the expert kernel's achieved HBM bandwidth on
activated-expert weight bytes, with the whole step's fraction beside it; `cpu_baseline` = the oracle on host
cores.  `--impl reference` times the oracle instead (it is the reference arm here: there is no reference code).

Other workloads: `--workload c3 | c4 --seqs N | paper` time the larger layer configurations the same way;
`--workload c5` runs the 48-layer MoE-only stack through the 4-step block loop for `--blocks` blocks, once with
TEAM's selection and once with vanilla top-k.  `--gpus N` without a launcher starts N replicas itself.
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
L2_NOTE = "inputs larger than L2: expert weights rotate over independent layers (GPU arm); the CPU oracle arm uses one layer"


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8000)
    ap.add_argument("--warmup", type=int, default=400)
    ap.add_argument("--impl", default="team", choices=["team", "reference"])
    ap.add_argument("--layers", type=int, default=None,
                    help="independent weight sets: cycled through by the layer workloads (default 8), depth of the c5 stack (default 48)")
    ap.add_argument("--flags", type=int, default=TEAM_FLAGS, help="0 vanilla, 1 DCD, 3 DCD|LAC")
    ap.add_argument("--no-graph", action="store_true", help="issue every step as separate calls (no CUDA graph)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="budget of the oracle baseline leg")
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c4", "paper", "c5", "decode", "attn"],
                    help="c2: the headline step (default); c3: 256 experts + shared, block 32; c4: c2 shape, --seqs x 4 "
                         "branches x 4; paper: c2 shape, block 32 x 4 branches in one group; c5: stack of c2 layers, block loop; "
                         "decode: the decode loop of blocks of 32 (acceptance, speculative branches, chained verification) "
                         "around the c2 layer, TEAM vs plain threshold decoding; attn: the attention half of delayed caching "
                         "(block 32 x 4 branches over a prefix of --prefix cached tokens)")
    ap.add_argument("--prefix", type=int, default=4096, help="cached tokens of earlier blocks in the attn workload")
    ap.add_argument("--seqs", type=int, default=1, help="sequences of the c4 batch sweep")
    ap.add_argument("--blocks", type=int, default=64, help="decoding blocks of the c5 stack run")
    ap.add_argument("--expert-kernel", default="auto", choices=["auto", "stream", "tile"],
                    help="auto: the library's choice by rows per call; stream: weight-streaming kernel; tile: tcgen05 grouped GEMMs")
    return ap.parse_args(argv)


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
    """(HBM GB/s, bf16 TFLOP/s burst, sustained, kind) from the measured-peaks file, else earlier measurements of the same GPU model."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops", 1590.0)), float(p.get("bf16_tflops_sustained", 1400.0)), "measured"
    return 6650.0, 1590.0, 1400.0, "fallback"


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


def workload_of(args):
    """(shape, workload string) of a layer workload."""
    from paper_2602_08404_b200 import workloads as W
    shape = {"c2": W.C2, "c3": W.C3, "c4": W.c4(args.seqs), "paper": W.paper_point(), "c5": W.C2}[args.workload]
    if args.workload == "c2" and args.flags == TEAM_FLAGS:
        return shape, WORKLOAD
    ns = shape.n_shared
    return shape, (f"{shape.name}: H{shape.hidden} E{shape.n_experts}{'+%d shared' % ns if ns else ''} top{shape.top_k} "
                   f"I{shape.inter} bf16, {shape.seqs} seq x {shape.branches} branches x block {shape.block} = {shape.rows} "
                   f"rows, {shape.n_steps} denoising steps, flags {args.flags}")


def config_of(args, shape, workload):
    """The workload's description: the same dictionary in the GPU arm and in the reference (oracle) arm."""
    return {"workload": workload, "flags": args.flags, "rows_presented": shape.rows, "l2": L2_NOTE,
            "parallelism": "replicas (one process per GPU, no exchange on the data path)"}


def oracle_leg(args, shape, weights_host, steps, budget_s, threads=None):
    """Times the oracle, as it stands, on the host cores over a bounded sample of the same workload.
    threads=None: whatever numpy's BLAS uses by default (all cores); threads=1: one thread."""
    from oracle import team_oracle as O
    from tests import _parity as P
    from threadpoolctl import threadpool_info, threadpool_limits
    ocfg = P.oracle_config(shape, args.flags)
    t_total, n = 0.0, 0
    y_prev = None
    with threadpool_limits(limits=threads):
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        while t_total < budget_s and n < 400:
            step = steps[n % len(steps)]
            t0 = time.perf_counter()
            y_prev, _ = O.moe_forward(ocfg, weights_host, step["x"], step["tok_state"], step["conf"], step["pos"],
                                      step["group"], step["branch"], y_prev=y_prev if n % len(steps) else None)
            t_total += time.perf_counter() - t0
            n += 1
    return {"value": shape.rows * n / t_total, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} layer-steps of the same schedule on one layer's weights ({t_total:.1f} s of CPU time)"}, \
        t_total / n


def run_reference(args):
    """The reference arm: the CPU oracle on the bench workload (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2602_08404_b200 import workloads as W
    shape, workload = workload_of(args)
    weights = W.make_weights(shape)
    steps = W.make_schedule(shape)
    budget = max(5.0, min(120.0, 0.05 * (args.steps + args.warmup)))
    cb, s_per_step = oracle_leg(args, shape, weights, steps, budget)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": 0,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": s_per_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_of(args, shape, workload),
            "cpu_baseline": cb,
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def init_device(args):
    """Process group (if launched as several ranks), device, library build.  Returns (world, rank, device)."""
    import torch
    import torch.distributed as dist
    from paper_2602_08404_b200 import build as build_mod
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
    return world, rank, torch.device("cuda", local_rank)


def run_layer(args):
    """The layer workloads (c2 headline, c3, c4, paper)."""
    import torch
    import torch.distributed as dist
    from paper_2602_08404_b200 import binding as B
    from paper_2602_08404_b200 import replicas as R_
    from paper_2602_08404_b200 import workloads as W

    world, rank, dev = init_device(args)
    shape, workload = workload_of(args)
    T, H, E, k, I = shape.rows, shape.hidden, shape.n_experts, shape.top_k, shape.inter
    ns = shape.n_shared
    steps_host = W.make_schedule(shape)                      # the scripted denoising steps, seeded
    n_sched = len(steps_host)
    R = args.layers or 8

    # R independent layers, generated on the device (seeded); layer 0 also goes to the host for the oracle leg
    layers, packed, tiles = [], [], []
    want_tiles = args.expert_kernel == "tile" or (args.expert_kernel == "auto" and T >= 96)
    want_classic = not want_tiles or args.expert_kernel == "stream"
    for r in range(R):
        wr, wg, wu, wd = W.device_layer_weights(shape, 1000 + r, dev)
        # the layouts the library reads; layer 0's row-major copies are kept for the oracle leg
        tiles.append(B.team_pack_w_tiles(wg, wu, wd) if want_tiles else (None, None))
        packed.append(B.team_pack_w_down(wd) if want_classic else None)
        keep = r == 0 or want_classic
        layers.append((wr, wg if keep else None, wu if keep else None, wd if r == 0 else None))
    cfg = B.make_config(H, E, k, I, ns, max_rows=T, max_groups=shape.seqs, dtype=B.TEAM_DTYPE_BF16, flags=args.flags,
                        tau_hot=shape.tau_hot, L_hot=shape.L_hot)
    ctxs = []
    for r in range(R):
        c = B.team_create(cfg)
        if want_classic:
            B.team_set_weights(c, *layers[r][:3], packed[r], *tiles[r])
        else:
            B.team_set_weights(c, layers[r][0], None, None, None, *tiles[r])
        if args.expert_kernel != "auto":
            B.team_debug_knob(c, B.TEAM_KNOB_EXPERT_KERNEL, 1 if args.expert_kernel == "stream" else 2)
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

    # CUDA graphs: one graph of whole cycles (up to 64 steps, no more than the timed region holds), and the remainder
    # of the timed region (steps % that), so that the timed region consists of graph replays only, whatever --steps
    # is, and a replay's launch gap is spread over many steps
    def capture(n):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(n):
                one_step(i)
        return g

    graph = tail_graph = None
    chunk = period * max(1, min(64 // period, args.steps // period))
    n_tail = args.steps % chunk
    if not args.no_graph:
        try:
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for i in range(period):
                    one_step(i)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = capture(chunk)
            tail_graph = capture(n_tail) if n_tail else None
        except Exception as e:                                   # report, and time plain launches instead
            print(f"[bench] CUDA graph capture failed ({e}); timing plain launches", file=sys.stderr)
            graph = tail_graph = None

    def run_steps(n):
        """Issues exactly n steps: whole graphs of `chunk` steps as replays, the remainder as one more replay (n %
        chunk == steps % chunk) or as plain calls."""
        if graph is None:
            for i in range(n):
                one_step(i)
            return n
        for _ in range(n // chunk):
            graph.replay()
        if n % chunk:
            if tail_graph is not None and n % chunk == n_tail:
                tail_graph.replay()
            else:
                for i in range(n % chunk):
                    one_step(i)
        return n

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(dev.index)
    with sampler:
        # ---- device-resident timing -----------------------------------------------------------------
        # Untimed, whatever --warmup says: every graph replayed at least twice, every context called, and at least
        # ~90 ms of the workload so that the clocks have settled (a first process on a cold GPU needs it).  Then the caller's warm-up steps.
        warm = 0
        for _ in range(2):
            warm += run_steps(chunk + n_tail)
        warm += run_steps(max(args.warmup, 3))
        warm += run_steps(chunk * max(0, (3000 - warm + chunk - 1) // chunk))
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
        n_roof = max(period, min(18 * period, 144))
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

        n_e2e = min(2000, max(args.steps, 400))      # the end-to-end leg has a step count of its own (printed): host timing needs a few hundred calls
        # on a stream of its own: the library records the step (copy in, kernels, copy out) as a graph, which the
        # legacy default stream cannot do
        e2e_stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(e2e_stream):
            # untimed: every context allocates its staging block and records its step on its first call, so every
            # context is called (twice) before the clock starts, whatever --warmup says
            e2e_warm = max(8 * period, min(args.warmup, 200))
            for i in range(e2e_warm):
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
    peak, tf_burst, tf_sustained, peak_kind = measured_peaks()
    # Where the whole step is ONE launch of the dominant kernel, the timed region is K back-to-back launches of it:
    # its average launch duration over the timed region is the step time (launch gaps included).  The event-bracketed
    # figure taken on plain launches is kept beside it (kernel_ms_isolated): there every launch pays its full launch
    # latency and cannot overlap its predecessor's tail, which the replayed graph allows.
    kernel_ms_isolated = kernel_ms
    if launches_per_step == 1 and graph is not None:
        kernel_ms = ms_per_step
    achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
    value = R_.whole_job_rate(T, ms_per_step)
    step_bytes = algo_bytes + 4 * E * H                           # + the router's weights
    step_frac = step_bytes / (ms_per_step * 1e-3) / 1e9 / peak
    tensor_tflops = mean_rows * (k + ns) * 6.0 * H * I / (kernel_ms * 1e-3) / 1e12
    kernel_name = B.team_expert_kernel_name(ctxs[0])

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": config_of(args, shape, workload),
        "run": {"layers_cycled": R, "weights_gb": R * (E + ns) * bytes_per_expert / 1e9, "cuda_graph": graph is not None, "graph_steps": chunk if graph is not None else 0,
                "steps_issued": issued, "warmup_issued": warm, "e2e_warmup_issued": e2e_warm,
                "rows_computed_mean": mean_rows, "activated_experts_mean": mean_act},
        "clocks": clocks,
        "e2e": {"value": R_.whole_job_rate(T, e2e_ms_per_step), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms_per_step, "steps": n_e2e},
        "gpu_launches": launches_per_step * issued,
        "activated_experts_per_s": R_.whole_job_rate(mean_act, ms_per_step),
        "rows_computed_per_s": R_.whole_job_rate(mean_rows, ms_per_step),
        "step_hbm_frac": step_frac,
        "roofline": {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                     "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_8TBs_nominal": achieved / 8000.0, "kernel_ms": kernel_ms,
                     "kernel_ms_isolated": kernel_ms_isolated,
                     "kernel_ms_from": "timed region (one launch per step)" if kernel_ms != kernel_ms_isolated or launches_per_step == 1 and graph is not None else "CUDA events around every launch",
                     "algorithmic_bytes_per_launch": algo_bytes, "launches_timed": tot_n,
                     # the whole step (router + selection + experts, graph replay) on its algorithmic bytes
                     "step_frac": step_frac, "step_frac_of_8TBs_nominal": step_bytes / (ms_per_step * 1e-3) / 8e12,
                     "step_bytes": step_bytes,
                     # DRAM read + write bytes per launch from the committed ncu capture, scaled to this run's mean
                     "traffic": traffic_per_launch(args, kernel_name, mean_act),
                     # the same launches as a contraction: 6 H I flops per token-slot (routed and shared)
                     "tensor_tflops": tensor_tflops, "tensor_frac_of_sustained": tensor_tflops / tf_sustained,
                     "tensor_frac_of_burst": tensor_tflops / tf_burst},
    }

    if rank == 0:
        if world == 1 and args.cpu_seconds > 0:
            weights_host = {n: t.float().cpu().numpy() for n, t in
                            zip(("w_router", "w_gate", "w_up", "w_down"), layers[0])}
            cb, _ = oracle_leg(args, shape, weights_host, steps_host, args.cpu_seconds * 0.75)
            one, _ = oracle_leg(args, shape, weights_host, steps_host, args.cpu_seconds * 0.25, threads=1)
            cb["single_thread"] = {"value": one["value"], "cores": one["cores"], "sample": one["sample"]}
            line["cpu_baseline"] = cb
        print(json.dumps(line))
    for c in ctxs:
        B.team_destroy(c)
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (read + write) per launch of the expert kernel at 16 activated experts, from the ncu capture whose
# summary is committed under profiles/ (None once the kernel has changed since the counters were taken).
TRAFFIC_AT_16_EXPERTS = {"k_experts_stream (fused step: router, selection and experts in one launch)": 152.13e6 + 3.40e6}


def traffic_per_launch(args, kernel_name, mean_act):
    t = TRAFFIC_AT_16_EXPERTS.get(kernel_name)
    return mean_act * t / 16.0 if (t is not None and args.workload == "c2") else None


def run_c5(args):
    """Config 5: a stack of SDAR-shaped MoE layers with residual adds, run through the 4-step denoising loop of
    `--blocks` decoding blocks, once with TEAM's selection (delayed caching + limited activation) and once with
    vanilla top-k.  A step here is one denoising step of the whole stack (all layers)."""
    import torch
    import torch.distributed as dist
    from paper_2602_08404_b200 import binding as B
    from paper_2602_08404_b200 import replicas as R_
    from paper_2602_08404_b200 import workloads as W
    import dataclasses

    world, rank, dev = init_device(args)
    shape = W.C2
    T, H, E, k, I = shape.rows, shape.hidden, shape.n_experts, shape.top_k, shape.inter
    L = args.layers or W.C5_LAYERS
    n_blocks = args.blocks
    bytes_per_expert = 3 * H * I * 2
    layers = []
    for l in range(L):
        wr, wg, wu, wd = W.device_layer_weights(shape, 5000 + l, dev)
        layers.append((wr, wg, wu, B.team_pack_w_down(wd)))
        del wd
    # every block has its own seeded schedule (hidden states, confidences); the acceptance pattern is the scripted one
    blocks = [W.make_schedule(shape, seed=shape.seed * 1000 + 29 + 7919 * b) for b in range(n_blocks)]
    n_sched = len(blocks[0])
    x_all = torch.stack([torch.stack([B.to_device(s["x"], B.TEAM_DTYPE_BF16, dev) for s in blk]) for blk in blocks])
    conf_all = torch.stack([torch.stack([torch.as_tensor(s["conf"]).to(dev) for s in blk]) for blk in blocks])
    st_static = [B.state_to_device(s, dev) for s in blocks[0]]      # states, positions, groups: the same in every block
    x_work = torch.zeros((T, H), dtype=torch.bfloat16, device=dev)
    y_dev = torch.zeros((T, H), dtype=torch.float32, device=dev)

    results = {}
    sampler = ClockSampler(dev.index)
    with sampler:
        for name, flags in (("team", TEAM_FLAGS), ("vanilla", 0)):
            cfg = B.make_config(H, E, k, I, 0, max_rows=T, max_groups=1, dtype=B.TEAM_DTYPE_BF16, flags=flags,
                                tau_hot=shape.tau_hot, L_hot=shape.L_hot)
            ctxs = []
            for l in range(L):
                c = B.team_create(cfg)
                B.team_set_weights(c, *layers[l])
                ctxs.append(c)

            def stack_step(s, n_act_out=None, bi=0):
                """One denoising step of the stack: x <- x + layer(x) on the computed rows, layer after layer."""
                for l, c in enumerate(ctxs):
                    out = None
                    if n_act_out is not None:
                        out = {"n_active": n_act_out[bi, s, l:l + 1], "n_rows_active": n_act_out[bi, s, L + l:L + l + 1]}
                    B.team_moe_forward(c, x_work, st_static[s], out, y_dev)
                    B.team_residual_add(c, x_work, y_dev, T)

            def load_block(b, s):
                x_work.copy_(x_all[b, s])
                st_static[s]["conf"].copy_(conf_all[b, s])

            # accounting pass (untimed): activated experts and computed rows of every (block, step, layer)
            counts = torch.zeros((n_blocks, n_sched, 2 * L), dtype=torch.int32, device=dev)
            for b in range(n_blocks):
                for s in range(n_sched):
                    load_block(b, s)
                    stack_step(s, counts, b)
            torch.cuda.synchronize()
            for c in ctxs:
                code, detail = B.team_read_status(c)
                if code != 0:
                    raise SystemExit(f"device status {code} detail {detail}")
            counts = counts.cpu().numpy().astype(np.int64)
            n_act, n_rows = counts[:, :, :L], counts[:, :, L:]
            x_final_check = float(x_work.float().abs().max())

            # one graph per denoising step of the stack (L layers: router, selection, experts, residual add each)
            graphs = []
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for s in range(n_sched):
                    load_block(0, s)
                    stack_step(s)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            for s in range(n_sched):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    stack_step(s)
                graphs.append(g)

            def run_blocks(nb):
                for b in range(nb):
                    for s in range(n_sched):
                        load_block(b, s)
                        graphs[s].replay()

            run_blocks(min(n_blocks, 4))                       # warm-up
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            run_blocks(n_blocks)
            e1.record()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            ms = R_.max_over_ranks(e0.elapsed_time(e1), dev)
            results[name] = dict(ms=ms, n_act=n_act, n_rows=n_rows, x_absmax=x_final_check)
            for c in ctxs:
                B.team_destroy(c)
    clocks = sampler.summary()

    peak, _, _, peak_kind = measured_peaks()
    stack_steps = n_blocks * n_sched

    def summarise(r):
        layer_steps = stack_steps * L
        act_total = float(r["n_act"].sum())
        bytes_total = act_total * bytes_per_expert + layer_steps * 4 * E * H
        return {"ms_total": r["ms"], "ms_per_stack_step": r["ms"] / stack_steps, "us_per_layer_step": r["ms"] * 1e3 / layer_steps,
                "rows_presented_per_s": R_.whole_job_rate(T * stack_steps, r["ms"]),
                "rows_computed_per_s": R_.whole_job_rate(float(r["n_rows"][:, :, 0].sum()), r["ms"]),
                "activated_experts_per_s": R_.whole_job_rate(act_total, r["ms"]),
                "activated_experts_per_layer_step": act_total / layer_steps,
                "step_frac": bytes_total / (r["ms"] * 1e-3) / 1e9 / peak,
                "step_frac_of_8TBs_nominal": bytes_total / (r["ms"] * 1e-3) / 8e12}

    team, vanilla = summarise(results["team"]), summarise(results["vanilla"])
    workload = (f"c5_stack: {L} x (H{H} E{E} top{k} I{I} bf16) MoE-only layers with residual adds, batch 1 x block {shape.block}, "
                f"{n_sched} denoising steps x {n_blocks} blocks, TEAM (DCD|LAC) vs vanilla top-k")
    line = {
        "metric": METRIC, "value": team["rows_presented_per_s"], "unit": UNIT, "n_gpus": world,
        "steps": stack_steps, "warmup": min(n_blocks, 4) * n_sched, "ms_per_step": team["ms_per_stack_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload, "flags": TEAM_FLAGS, "rows_presented": T,
                   "l2": f"inputs larger than L2: {L} layers of weights ({L * E * bytes_per_expert / 1e9:.1f} GB) are walked once per denoising step",
                   "parallelism": "replicas (one process per GPU, no exchange on the data path)"},
        "note": "a step is one denoising step of the whole stack; value counts rows presented to the stack per second "
                "(each row passes through every layer)",
        "clocks": clocks, "team": team, "vanilla": vanilla,
        "vanilla_over_team_time": vanilla["ms_total"] / team["ms_total"],
        "paper_context": "the paper reports up to 2.2x end-to-end decoding speed-up of TEAM over the vanilla model on one "
                         "A100 80GB (whole SDAR 30B-A3B model incl. attention and speculative branches); not comparable",
        "roofline": {"bound": "hbm", "kernel": "whole stack step (router, selection, experts, residual add per layer)",
                     "achieved": team["step_frac"] * peak, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                     "frac": team["step_frac"], "traffic": None},
        "gpu_launches": stack_steps * L * 4,
    }
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_decode(args):
    """The decode loop of one sequence, block by block (Eq. 2-3, Sec. 4.2 / 5.4), around one SDAR-shaped MoE layer:
    every forward pass is team_seh_step (acceptance, chained verification, next candidates, rows) followed by
    team_moe_forward on those rows.  The language-model head is a seeded script (there is no model here); the hidden
    states are the synthetic generator's.  TEAM = 4 speculative branches + delayed caching + limited activation;
    vanilla = one branch, plain top-k.  Reports TPF (accepted tokens per forward pass), APF (activated experts per
    forward pass of this layer) and APT = APF / TPF, the quantities of the paper's Table 1, and the time per pass."""
    import torch
    from paper_2602_08404_b200 import binding as B
    from paper_2602_08404_b200 import workloads as W
    import dataclasses

    world, rank, dev = init_device(args)
    base = W.paper_point()                                     # block 32, L_hot 3
    L, H, E, k, I = base.block, base.hidden, base.n_experts, base.top_k, base.inter
    n_blocks, tau, max_steps = args.blocks, 0.95, 96
    R = args.layers or 4
    layers = []
    for r in range(R):
        wr, wg, wu, wd = W.device_layer_weights(base, 1000 + r, dev)
        layers.append((wr, wg, wu, B.team_pack_w_down(wd), *B.team_pack_w_tiles(wg, wu, wd)))
        del wd
    scripts = [W.make_decode_script(1, L, max_steps, seed=900 + b) for b in range(n_blocks)]
    results = {}
    sampler = ClockSampler(dev.index)
    with sampler:
        for name, nb, flags in (("team", 4, TEAM_FLAGS), ("vanilla", 1, 0)):
            shape = dataclasses.replace(base, branches=nb)
            T = shape.rows
            xs = [B.to_device(st["x"], B.TEAM_DTYPE_BF16, dev) for st in W.make_schedule(shape)]      # hidden states, cycled
            cfg = B.make_config(H, E, k, I, 0, max_rows=T, max_groups=1, dtype=B.TEAM_DTYPE_BF16, flags=flags,
                                tau_hot=base.tau_hot, L_hot=base.L_hot)
            ctxs = []
            for r in range(R):
                c = B.team_create(cfg)
                B.team_set_weights(c, *layers[r])
                ctxs.append(c)
            state, rows = B.seh_alloc(1, L, nb, dev)
            y = torch.zeros((T, H), dtype=torch.float32, device=dev)
            pd = [(torch.as_tensor(p[:, :, :nb]).to(dev).contiguous(), torch.as_tensor(c[:, :, :nb]).to(dev).contiguous())
                  for p, c in scripts]
            n_act = torch.zeros((n_blocks * max_steps,), dtype=torch.int32, device=dev)

            def run(count_only):
                """One pass over all blocks; returns forward passes per block (count_only: the glue alone, with a
                host check after every step; otherwise exactly the counted passes, no host synchronisation)."""
                fwd, i = [], 0
                for b in range(n_blocks):
                    B.team_seh_step(1, L, nb, tau, state, None, None, rows)
                    n = 0
                    for s in range(max_steps if count_only else passes[b]):
                        if count_only:
                            if not bool((state["state"] == 0).any()):
                                break
                        else:
                            out = {"n_active": n_act[i:i + 1]}
                            B.team_moe_forward(ctxs[i % R], xs[s % len(xs)], rows, out, y)
                        B.team_seh_step(1, L, nb, tau, state, pd[b][0][s], pd[b][1][s], rows)
                        n += 1
                        i += 1
                    fwd.append(n)
                return fwd

            passes = run(True)
            run(False)                                        # warm-up, and the activated experts of every pass
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            run(False)
            e1.record()
            torch.cuda.synchronize()
            total = sum(passes)
            launches = (B.team_last_launch_count(ctxs[0]) + 1) * total        # the layer's kernels + the glue kernel, per pass
            apf = float(n_act[:total].float().mean())
            results[name] = {"forward_passes": total, "decoded_tokens": n_blocks * L, "TPF": n_blocks * L / total, "APF": apf,
                             "APT": apf * total / (n_blocks * L), "rows_per_pass": T, "gpu_launches": launches, "us_per_pass": e0.elapsed_time(e1) * 1e3 / total,
                             "decoded_tokens_per_s_this_layer": n_blocks * L / (e0.elapsed_time(e1) * 1e-3)}
            for c in ctxs:
                B.team_destroy(c)
    t, v = results["team"], results["vanilla"]
    line = {"metric": METRIC, "value": t["rows_per_pass"] / (t["us_per_pass"] * 1e-6), "unit": UNIT, "n_gpus": world,
            "steps": t["forward_passes"], "warmup": t["forward_passes"], "ms_per_step": t["us_per_pass"] * 1e-3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"decode loop: {n_blocks} blocks of {L}, tau {tau}, scripted language-model head; c2 layer "
                                   f"(H{H} E{E} top{k} I{I}); TEAM = 4 branches + DCD|LAC vs vanilla = 1 branch, top-k",
                       "flags": TEAM_FLAGS, "rows_presented": t["rows_per_pass"], "l2": L2_NOTE,
                       "parallelism": "replicas (one process per GPU, no exchange on the data path)"},
            "clocks": sampler.summary(), "team": t, "vanilla": v,
            "decode_speedup_this_layer": t["decoded_tokens_per_s_this_layer"] / v["decoded_tokens_per_s_this_layer"],
            "paper_context": "Table 1 (SDAR 30B-A3B, one A100 80GB, real model): TPF 3.14 -> 5.00, APF 54.99 -> 34.48, APT 17.66 -> 6.92, "
                             "speed-up 1.94x on average; a scripted head and synthetic hidden states stand in here",
            "gpu_launches": t["gpu_launches"]}
    if rank == 0:
        print(json.dumps(line))


def run_attn(args):
    """The attention half of delayed caching (Sec. 4.1) on an SDAR-like attention shape: 32 query heads, 4 key/value
    heads, head size 128, one sequence, block 32 x 4 branches, a prefix of --prefix cached tokens.  Successive calls
    rotate over --layers independent KV caches so that keys and values come from HBM.  Algorithmic bytes per call =
    prefix and in-block K/V read once + q + fresh k/v + output."""
    import torch
    from paper_2602_08404_b200 import binding as B
    from paper_2602_08404_b200 import workloads as W

    world, rank, dev = init_device(args)
    shape = W.paper_point()
    S, Bn, L, T = 1, shape.branches, shape.block, shape.rows
    Hq, Hkv, d, P = 32, 4, 128, args.prefix
    R = args.layers or 16
    steps = W.make_schedule(shape)
    st = [B.state_to_device(s, dev) for s in steps]
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    rnd = lambda *sh: torch.randn(sh, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    caches = [(rnd(S, P, Hkv, d), rnd(S, P, Hkv, d), rnd(S, L, Hkv, d), rnd(S, L, Hkv, d)) for _ in range(R)]
    q, k, v = rnd(T, Hq, d), rnd(T, Hkv, d), rnd(T, Hkv, d)
    plen = torch.full((S,), P, dtype=torch.int32, device=dev)
    out = torch.zeros((T, Hq, d), dtype=torch.float32, device=dev)
    res = {}
    sampler = ClockSampler(dev.index)
    with sampler:
        for name, flags in (("delayed_caching", 1), ("recompute_all", 0)):
            cfg = B.team_attn_config(Hq, Hkv, d, L, S, Bn, P, flags)

            def call(i):
                kp, vp, kb, vb = caches[i % R]
                rc = B.team_block_attention(cfg, st[i % len(st)], q, k, v, kp, vp, plen, kb, vb, out)
                if rc != 0:
                    raise SystemExit(f"team_block_attention returned {rc}")

            for i in range(max(3, R)):
                call(i)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(R * len(st)):
                    call(i)
            n = R * len(st)
            for _ in range(3):
                g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(1, args.steps // n)
            e0.record()
            for _ in range(reps):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / (reps * n)
            comp = np.mean([(s["tok_state"] != 2).sum() if flags else T for s in steps])
            bytes_ = 2 * (P + L) * Hkv * d * 2 + comp * Hq * d * (2 + 4) + 2 * T * Hkv * d * 2
            flops = 4.0 * comp * Hq * (P + L) * d          # q k^T and p v, 2 flops per multiply-add
            res[name] = {"us_per_call": us, "rows_computed_mean": float(comp), "algorithmic_bytes": float(bytes_),
                         "hbm_frac": bytes_ / (us * 1e-6) / 1e9 / measured_peaks()[0],
                         "algorithmic_flops": flops, "tensor_tflops": flops / (us * 1e-6) / 1e12}
    t = res["delayed_caching"]
    line = {"metric": METRIC, "value": T / (t["us_per_call"] * 1e-6), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": 3, "ms_per_step": t["us_per_call"] * 1e-3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"attention half of delayed caching: {Hq} query / {Hkv} kv heads x {d}, block {L} x {Bn} branches, "
                                   f"prefix {P}", "flags": 1, "rows_presented": T,
                       "l2": f"inputs larger than L2: KV caches rotate over {R} layers", "parallelism": "replicas"},
            "clocks": sampler.summary(), "delayed_caching": t, "recompute_all": res["recompute_all"],
            # a contraction: at this shape the flops take longer on the tensor roof than the bytes on the HBM roof
            "roofline": {"bound": "tensor", "kernel": "k_block_attention", "achieved": t["tensor_tflops"],
                         "peak": measured_peaks()[2], "peak_kind": "of " + measured_peaks()[3] + " (bf16 sustained)",
                         "unit": "TFLOP/s", "frac": t["tensor_tflops"] / measured_peaks()[2], "hbm_frac": t["hbm_frac"],
                         "traffic": None},
            "gpu_launches": 2 * args.steps}
    if rank == 0:
        print(json.dumps(line))


def main(argv=None):
    args = parse_args(argv)
    from paper_2602_08404_b200 import replicas as R_
    if R_.needs_launcher(args.gpus):
        # --gpus N without a launcher: start the N replicas ourselves (one process per GPU), pass their output through
        raise SystemExit(R_.run_under_launcher(os.path.abspath(__file__), sys.argv[1:] if argv is None else argv, args.gpus))
    if args.impl == "reference":
        return run_reference(args)
    if args.workload == "c5":
        return run_c5(args)
    if args.workload == "decode":
        return run_decode(args)
    if args.workload == "attn":
        return run_attn(args)
    return run_layer(args)


if __name__ == "__main__":
    main()
