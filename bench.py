"""Benchmark of the E2-TTT chunk-parallel fast-weight update on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]

A step is one pass of the whole hot path (e2ttt_chunk_fwd over every chunk of every sequence) on one
batch of seeded synthetic inputs.  Default workload: the 1.3B-layer shape (B=4, H=16, d=128, h=512,
L=4096, C=64, bf16 I/O, GELU-MLP fast weights), forward.  One JSON line is printed by rank 0.

  value     layer tokens/s (B*L per call / device time), inputs resident in HBM
  e2e       the same metric through the C ABI with HOST buffers: pinned-host -> device copies of all
            inputs and device -> host copies of all results inside the timed region
  roofline  for the forward kernel: algorithmic GEMM flop per launch / CUDA-event time per launch
            against the measured bf16 dense peak of this machine (MEASURED_PEAKS.json)
  cpu_baseline  the fp64 oracle, as it stands, timed on the host cores over a bounded sample

`--impl reference` times the oracle itself (there is no other reference implementation of this path).
With N > 1 (torchrun) every rank runs the same workload on its own seeded batch: the path shards over
(batch, head) with no exchange, so scaling is weak and the only collectives are the timing barrier and
a MAX over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_21308_b200 import inputs  # noqa: E402

METRIC = "e2ttt_layer_fwd_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per forward launch from the committed ncu capture
# (profiles/): set once a capture of the current kernel exists, else null.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 338.5e6  # profiles/tc_fwd_kernel_config2.md: 238.2 MB read + 92.9 MB written


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    return dict(FALLBACK_PEAKS, _source="fallback")


def flops_per_token_head(r: inputs.Recipe, backward: bool = False) -> float:
    """GEMM flop the method needs per token and head: 9 (MLP) or 13 (SwiGLU) products of 2*d*h forward,
    23 more units for the reverse pass (5 of them recomputed forward products)."""
    units = 9 if r.kind == inputs.KIND_MLP else 13
    f = units * 2.0 * r.d * r.h
    if backward:
        f += 23 * 2.0 * r.d * r.h
    return f


def bytes_per_call(r: inputs.Recipe) -> float:
    s = 2 if r.io == "bf16" else 4
    nm = len(inputs.mat_shapes(r.kind, r.d, r.h))
    n = r.B * r.H
    return n * r.L * (4 * r.d * s + 12) + n * 4 * nm * r.d * r.h * 4


class ClockSampler:
    """nvidia-smi sampled every 200 ms while the timed region runs (read-only queries)."""

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows:
            try:
                sm.append(float(row[0]))
                mx.append(float(row[1]))
            except (ValueError, IndexError):
                continue
            for n, val in zip(names, row[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "samples_under_load": len(sm), "reasons": sorted(reasons)}


def cpu_oracle_rate(r: inputs.Recipe, budget_heads: int | None = None, tokens: int = 512):
    """Time the oracle (untouched) on a bounded sample: `cores` heads x `tokens` tokens of the workload."""
    from oracle import oracle
    cores = oracle.max_threads()
    n_heads = budget_heads or max(cores, 1)
    rs = inputs.Recipe(**{**r.__dict__, "L": min(tokens, r.L), "heads": list(range(min(n_heads, r.B * r.H)))})
    x = inputs.generate(rs)
    t0 = time.perf_counter()
    oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], None, r.C, r.kind, threads=cores)
    dt = time.perf_counter() - t0
    token_heads = len(rs.heads) * rs.L
    return {"value": token_heads / r.H / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(rs.heads)} heads x {rs.L} tokens of the workload, fp64, forward; "
                      f"layer tokens/s = token-heads/s / H", "seconds": dt}


def run_reference(args, r):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for i in range(args.warmup + args.steps):
        res = cpu_oracle_rate(r)  # the same bounded sample as the cpu_baseline leg of the other arm
        if i >= args.warmup:
            vals.append(res)
    dt = float(np.mean([v["seconds"] for v in vals]))
    value = float(np.mean([v["value"] for v in vals]))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(r),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": vals[0]["cores"], "kind": "oracle",
                             "sample": vals[0]["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def shard_recipe(r, rank: int):
    """Rank `rank`'s share of an N-GPU run: the same shapes, its own seeded batch (weak scaling, no exchange)."""
    return inputs.Recipe(**{**r.__dict__, "seed": r.seed + rank})


def whole_job_value(world: int, tokens_per_rank: int, ms_max_over_ranks: float) -> float:
    """Whole-job throughput: the tokens all ranks processed / the slowest rank's device time."""
    return world * tokens_per_rank / (ms_max_over_ranks * 1e-3)


def max_over_ranks(ms: float, dist, device) -> float:
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gates_text(r):
    """The gate recipe of the run, as the JSON line states it."""
    tau = "" if r.tau == 1.0 else f"^(1/{r.tau:g})"
    regime = "paper regime (eta_base 0.01, tau 32, alpha_base 0.1): " if (r.eta_base, r.tau, r.alpha_base) == (0.01, 32.0, 0.1) else ""
    return (f"{regime}eta={r.eta_base:g}*sigmoid(N(0,1)), beta=sigmoid(N(1,1)){tau}, "
            f"gamma=1-eta*{r.alpha_base:g}*sigmoid(N(3,1))")


def workload_config(r):
    kind = "mlp_gelu" if r.kind == inputs.KIND_MLP else "swiglu"
    return {"workload": f"e2ttt_chunk_fwd B={r.B} H={r.H} L={r.L} d={r.d} h={r.h} C={r.C} {kind} {r.io} I/O",
            "B": r.B, "H": r.H, "L": r.L, "d": r.d, "h": r.h, "C": r.C, "kind": kind, "io": r.io,
            "gates": gates_text(r), "seed": r.seed,
            "l2": "inputs larger than L2: q,k,v,o and states of one call exceed 126 MB"}


def run_ours(args, r):
    import torch
    import torch.distributed as dist
    from paper_2608_21308_b200 import binding as E

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    x = inputs.generate(shard_recipe(r, rank))
    N = r.B * r.H
    iod = torch.float32 if r.io == "f32" else torch.bfloat16
    impl = {"auto": E.E2TTT_IMPL_AUTO, "fused": E.E2TTT_IMPL_TCGEN05, "tiled": E.E2TTT_IMPL_TILED, "simt": E.E2TTT_IMPL_SIMT}[args.kernel]
    p = E.make_params(r.B, r.H, r.L, r.d, r.h, r.C, r.kind, E.E2TTT_F32 if r.io == "f32" else E.E2TTT_BF16, 1e-5, impl)
    s4, s3 = (r.B, r.H, r.L, r.d), (r.B, r.H, r.L)
    shapes = inputs.mat_shapes(r.kind, r.d, r.h)
    host = {n: torch.from_numpy(x[n]).to(iod).view(s4).pin_memory() for n in ("q", "k", "v")}
    host.update({n: torch.from_numpy(x[n]).view(s3).pin_memory() for n in ("eta", "beta", "gamma")})
    hostW = [torch.from_numpy(w).view((r.B, r.H) + s).pin_memory() for w, s in zip(x["W"], shapes)]
    devt = {n: t.to(dev) for n, t in host.items()}
    W0 = [w.to(dev) for w in hostW]
    o = torch.empty(s4, dtype=iod, device=dev)
    Wf = [torch.empty_like(w) for w in W0]
    Mf = [torch.empty_like(w) for w in W0]
    ws = torch.empty((E.e2ttt_workspace_bytes_normed if args.post_norm else E.e2ttt_workspace_bytes)(p, 0),
                     dtype=torch.uint8, device=dev)
    # --post-norm: targets = the row norms of the initial fast weights, as a model would set them
    row_norm = [w.float().pow(2).sum(-1).sqrt().contiguous() for w in W0] if args.post_norm else None
    host_o = torch.empty(s4, dtype=iod).pin_memory()
    host_Wf = [torch.empty_like(w).pin_memory() for w in hostW]
    host_Mf = [torch.empty_like(w).pin_memory() for w in hostW]
    stream = torch.cuda.current_stream()

    def step():
        if args.post_norm:
            E.e2ttt_chunk_fwd_normed(p, devt["q"], devt["k"], devt["v"], devt["eta"], devt["beta"], devt["gamma"], W0, None,
                                     row_norm, 1e-5, o, Wf, Mf, ws, 0, stream)
        else:
            E.e2ttt_chunk_fwd(p, devt["q"], devt["k"], devt["v"], devt["eta"], devt["beta"], devt["gamma"], W0, None, o,
                              Wf, Mf, ws, 0, stream)

    # End to end: every step copies its inputs from pinned host memory and its results back.  The three legs run on
    # three streams over two sets of device buffers, so step i+1's upload and step i-1's download overlap step i's
    # kernel (the copy engines of the two directions are independent); every step still moves all of its bytes.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    sets = []
    for _ in range(2):
        sets.append(dict(t={n: torch.empty_like(v) for n, v in devt.items()}, W0=[torch.empty_like(w) for w in W0],
                         o=torch.empty_like(o), Wf=[torch.empty_like(w) for w in W0], Mf=[torch.empty_like(w) for w in W0],
                         ws=torch.empty_like(ws), ready=torch.cuda.Event(), computed=torch.cuda.Event(),
                         drained=torch.cuda.Event()))

    def run_e2e(n_steps):
        s_in.wait_stream(stream)
        s_out.wait_stream(stream)
        for i in range(n_steps):
            b = sets[i % 2]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(b["computed"])      # the kernel of step i-2 has read this set's inputs
                for n in host:
                    b["t"][n].copy_(host[n], non_blocking=True)
                for wd, wh in zip(b["W0"], hostW):
                    wd.copy_(wh, non_blocking=True)
                b["ready"].record(s_in)
            stream.wait_event(b["ready"])
            if i >= 2:
                stream.wait_event(b["drained"])          # step i-2's results have left this set's output buffers
            t = b["t"]
            if args.post_norm:
                E.e2ttt_chunk_fwd_normed(p, t["q"], t["k"], t["v"], t["eta"], t["beta"], t["gamma"], b["W0"], None, row_norm,
                                         1e-5, b["o"], b["Wf"], b["Mf"], b["ws"], 0, stream)
            else:
                E.e2ttt_chunk_fwd(p, t["q"], t["k"], t["v"], t["eta"], t["beta"], t["gamma"], b["W0"], None, b["o"],
                                  b["Wf"], b["Mf"], b["ws"], 0, stream)
            b["computed"].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(b["computed"])
                host_o.copy_(b["o"], non_blocking=True)
                for a, c in zip(host_Wf, b["Wf"]):
                    a.copy_(c, non_blocking=True)
                for a, c in zip(host_Mf, b["Mf"]):
                    a.copy_(c, non_blocking=True)
                b["drained"].record(s_out)
        stream.wait_stream(s_out)

    def timed_e2e(n_steps):
        run_e2e(2)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        run_e2e(n_steps)
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1) / n_steps
        if world > 1:
            ms = max_over_ranks(ms, dist, dev)
        return ms

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup, preroll_s):
        """W warm-up steps, then an untimed pre-roll of the same step that keeps the GPU under this load for
        `preroll_s` seconds (the 200 ms clock sampler needs a steady state to look at; a 20 ms region would give it one
        sample), then EXACTLY `steps` timed steps: one event pair around all of them (the reported mean) and one pair
        per step (the median)."""
        for _ in range(warmup):
            fn()
        barrier()
        t_end = time.perf_counter() + preroll_s
        n_pre = 0
        while time.perf_counter() < t_end:
            for _ in range(8):
                fn()
            n_pre += 8
            stream.synchronize()
        barrier()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record(stream)
        for i in range(steps):
            fn()
            ev[i + 1].record(stream)
        barrier()
        ms = ev[0].elapsed_time(ev[steps]) / steps
        per_call = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(steps))
        med = per_call[steps // 2]
        if world > 1:
            ms = max_over_ranks(ms, dist, dev)
            med = max_over_ranks(med, dist, dev)
        return ms, med, n_pre

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms, ms_median, n_preroll = timed(step, args.steps, args.warmup, args.preroll)
    clocks = sampler.stop() if rank == 0 else None
    # the timed calls must have run clean: device status 0 (no bounded wait gave up) and finite outputs
    status = E.e2ttt_device_status(ws, stream)
    finite = bool(torch.isfinite(o.float()).all().item()) and all(bool(torch.isfinite(w).all().item()) for w in Wf + Mf)
    if status != 0 or not finite:
        raise SystemExit(f"bench: the timed calls did not run clean (device status {status}, finite outputs {finite})")
    ms_e2e = timed_e2e(max(4, args.steps))

    if rank == 0:
        pk = peaks()
        tokens = r.B * r.L
        flop = flops_per_token_head(r) * N * r.L
        t_tc = flop / (pk["bf16_tflops"] * 1e12)
        t_hbm = bytes_per_call(r) / (pk["hbm_gbs"] * 1e9)
        bound = "tensor" if t_tc >= t_hbm else "hbm"
        if bound == "tensor":
            achieved, peak, unit = flop / (ms * 1e-3) / 1e12, pk["bf16_tflops"], "TFLOP/s"
        else:
            achieved, peak, unit = bytes_per_call(r) / (ms * 1e-3) / 1e9, pk["hbm_gbs"], "GB/s"
        h2d = sum(t.numel() * t.element_size() for t in host.values()) + sum(w.numel() * 4 for w in hostW)
        d2h = host_o.numel() * host_o.element_size() + 2 * sum(w.numel() * 4 for w in hostW)
        line = {
            "metric": METRIC, "value": whole_job_value(world, tokens, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "ms_per_step_median": ms_median,
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if r.io == "bf16" else "f64",
            "data": "synthetic",
            "timing": f"CUDA events on the launch stream; {args.warmup} warm-up steps, {n_preroll} untimed pre-roll steps "
                      f"(~{args.preroll:g} s of the same load, so the clock samples describe the timed region's steady state), "
                      f"then exactly {args.steps} timed steps; device status 0 and finite outputs checked afterwards",
            "config": dict(workload_config(r), kernel_family=args.kernel, **({"post_chunk_norm": "rows of every W_i rescaled to the row norms of W_init after each chunk (any-shape kernels)"} if args.post_norm else {})),
            "e2e": {"value": whole_job_value(world, tokens, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e,
                    "how": "per step: inputs and initial state from pinned host memory, outputs and final state back; upload, kernel and download of consecutive steps overlap on three streams"},
            "gpu_launches": args.steps,
            "clocks": clocks,
            "roofline": {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
                         "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH if args.config == 2 else None,
                         "peak_source": pk["_source"],
                         "kernel": "forward kernel (one launch per step)",
                         "flop_per_launch": flop, "bytes_per_launch": bytes_per_call(r),
                         "frac_of_sustained_peak": (flop / (ms * 1e-3) / 1e12) / pk["bf16_tflops_sustained"]},
        }
        if world == 1 and not args.no_cpu:
            line["cpu_baseline"] = {k: v for k, v in cpu_oracle_rate(r).items() if k != "seconds"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_fwd_bwd(args, r):
    """Optional second workload (--backward): one step = e2ttt_chunk_fwd(save_states=1) + e2ttt_chunk_bwd on the same
    batch (both networks).  The line names the kernels that ran."""
    import torch
    from paper_2608_21308_b200 import binding as E

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    x = inputs.generate(r, with_d_o=True)
    N = r.B * r.H
    iod = torch.float32 if r.io == "f32" else torch.bfloat16
    p = E.make_params(r.B, r.H, r.L, r.d, r.h, r.C, r.kind, E.E2TTT_F32 if r.io == "f32" else E.E2TTT_BF16, 1e-5,
                      E.E2TTT_IMPL_AUTO, args.ckpt_every)
    s4, s3 = (r.B, r.H, r.L, r.d), (r.B, r.H, r.L)
    shapes = inputs.mat_shapes(r.kind, r.d, r.h)
    host = {n: torch.from_numpy(x[n]).to(iod).view(s4).pin_memory() for n in ("q", "k", "v", "d_o")}
    host.update({n: torch.from_numpy(x[n]).view(s3).pin_memory() for n in ("eta", "beta", "gamma")})
    hostW = [torch.from_numpy(w).view((r.B, r.H) + s).pin_memory() for w, s in zip(x["W"], shapes)]
    t = {n: v.to(dev) for n, v in host.items()}
    W0 = [w.to(dev) for w in hostW]
    o = torch.empty(s4, dtype=iod, device=dev)
    Wf = [torch.empty_like(w) for w in W0]
    Mf = [torch.empty_like(w) for w in W0]
    dq, dk, dv = (torch.empty(s4, dtype=iod, device=dev) for _ in range(3))
    de, db, dg = (torch.empty(s3, dtype=torch.float32, device=dev) for _ in range(3))
    dW = [torch.empty_like(w) for w in W0]
    dM = [torch.empty_like(w) for w in W0]
    ws = torch.empty(E.e2ttt_workspace_bytes(p, 1), dtype=torch.uint8, device=dev)
    hout = [torch.empty(s4, dtype=iod).pin_memory() for _ in range(4)]
    stream = torch.cuda.current_stream()

    def step():
        E.e2ttt_chunk_fwd(p, t["q"], t["k"], t["v"], t["eta"], t["beta"], t["gamma"], W0, None, o, Wf, Mf, ws, 1, stream)
        E.e2ttt_chunk_bwd(p, t["q"], t["k"], t["v"], t["eta"], t["beta"], t["gamma"], W0, None, t["d_o"], None, None,
                          dq, dk, dv, de, db, dg, dW, dM, ws, 1, stream)

    def step_e2e():
        for n in host:
            t[n].copy_(host[n], non_blocking=True)
        step()
        for a, b in zip(hout, (o, dq, dk, dv)):
            a.copy_(b, non_blocking=True)

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    sampler = ClockSampler(0)
    sampler.start()
    ms = timed(step, args.steps, args.warmup)
    clocks = sampler.stop()
    ms_e2e = timed(step_e2e, max(1, args.steps // 2), 1)
    pk = peaks()
    tokens = r.B * r.L
    flop = flops_per_token_head(r, backward=True) * N * r.L
    cfg = workload_config(r)
    cfg["workload"] = cfg["workload"].replace("e2ttt_chunk_fwd", "e2ttt_chunk_fwd(save_states) + e2ttt_chunk_bwd")
    cfg["path"] = "fused tensor-core forward writing chunk-start states where it serves the shape, any-shape backward with tcgen05 GEMMs"
    cfg["ckpt_every"] = args.ckpt_every
    cfg["workspace_bytes"] = ws.numel()
    nseg = -(-(r.L // r.C) // args.ckpt_every) if args.ckpt_every >= 2 else 0
    line = {"metric": "e2ttt_layer_fwd_bwd_tokens_per_s", "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if r.io == "bf16" else "f64", "data": "synthetic", "config": cfg,
            "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": sum(v.numel() * v.element_size() for v in host.values()),
                    "d2h_bytes_per_step": sum(v.numel() * v.element_size() for v in hout), "ms_per_step": ms_e2e},
            "gpu_launches": (1 + max(1, 2 * nseg)) * args.steps, "clocks": clocks,
            "roofline": {"bound": "tensor", "achieved": flop / (ms * 1e-3) / 1e12, "peak": pk["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": flop / (ms * 1e-3) / 1e12 / pk["bf16_tflops"], "traffic": None,
                         "peak_source": pk["_source"], "flop_per_step": flop}}
    print(json.dumps(line))


def run_decode(args, r):
    """Optional third workload (--decode): one step = e2ttt_apply for ONE new token of every sequence (the decode path
    between chunk boundaries).  HBM-bound: the step reads every sequence's fast weights once.  The weights of one
    step fit in L2, so the steps rotate over enough independent state copies to exceed it, as the layers of a model do."""
    import torch
    from paper_2608_21308_b200 import binding as E

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    rr = inputs.Recipe(**{**r.__dict__, "L": 1})
    x = inputs.generate(rr)
    N = r.B * r.H
    iod = torch.float32 if r.io == "f32" else torch.bfloat16
    p = E.make_params(r.B, r.H, 1, r.d, r.h, 1, r.kind, E.E2TTT_F32 if r.io == "f32" else E.E2TTT_BF16, 1e-5,
                      E.E2TTT_IMPL_AUTO)
    shapes = inputs.mat_shapes(r.kind, r.d, r.h)
    s4 = (r.B, r.H, 1, r.d)
    host_q = torch.from_numpy(x["q"]).to(iod).view(s4).pin_memory()
    host_o = torch.empty(s4, dtype=iod).pin_memory()
    q = host_q.to(dev)
    o = torch.empty_like(q)
    state_bytes = sum(4 * N * a * b for a, b in shapes)
    copies = max(2, int(3 * 126e6 // state_bytes) + 1)
    Ws = []
    for c in range(copies):
        Ws.append([torch.from_numpy(w).view((r.B, r.H) + s).to(dev) * (1.0 + 0.01 * c) for w, s in zip(x["W"], shapes)])
    stream = torch.cuda.current_stream()
    it = [0]

    def step(st=None):
        E.e2ttt_apply(p, q, Ws[it[0] % copies], o, st if st is not None else stream)
        it[0] += 1

    def step_e2e():
        q.copy_(host_q, non_blocking=True)
        step()
        host_o.copy_(o, non_blocking=True)

    # A step is a ~10 us kernel: launched one by one from Python the host, not the GPU, sets the pace.  So one pass
    # over the state copies is captured in a CUDA graph (the library call only enqueues a kernel) and replayed.
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(copies):
            step(torch.cuda.current_stream())
    replays = max(1, -(-max(args.steps, 50) // copies))
    steps = replays * copies

    def timed_graph():
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(replays):
            graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    def timed(fn, n, warmup):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    sampler = ClockSampler(0)
    sampler.start()
    ms = timed_graph()
    clocks = sampler.stop()
    ms_eager = timed(step, steps, 3)
    ms_e2e = timed(step_e2e, steps, 3)

    # the other half of decoding: once C tokens have accumulated, e2ttt_chunk_fwd over them moves the state on
    C = r.C
    rc = inputs.Recipe(**{**r.__dict__, "L": C})
    xc = inputs.generate(rc)
    pc = E.make_params(r.B, r.H, C, r.d, r.h, C, r.kind, E.E2TTT_F32 if r.io == "f32" else E.E2TTT_BF16, 1e-5,
                       E.E2TTT_IMPL_AUTO)
    sc4, sc3 = (r.B, r.H, C, r.d), (r.B, r.H, C)
    cq, ck, cv = (torch.from_numpy(xc[n]).to(iod).view(sc4).to(dev) for n in ("q", "k", "v"))
    ce, cb, cg = (torch.from_numpy(xc[n]).view(sc3).to(dev) for n in ("eta", "beta", "gamma"))
    co = torch.empty_like(cq)
    Wn = [torch.empty_like(w) for w in Ws[0]]
    Mn = [torch.empty_like(w) for w in Ws[0]]
    wsc = torch.empty(E.e2ttt_workspace_bytes(pc, 0), dtype=torch.uint8, device=dev)
    iu = [0]

    def update():
        E.e2ttt_chunk_fwd(pc, cq, ck, cv, ce, cb, cg, Ws[iu[0] % copies], None, co, Wn, Mn, wsc, 0, stream)
        iu[0] += 1

    ms_update = timed(update, max(20, copies), 3)
    pk = peaks()
    io_bytes = 2 * N * r.d * (2 if r.io == "bf16" else 4)
    nbytes = state_bytes + io_bytes
    kind = "mlp_gelu" if r.kind == inputs.KIND_MLP else "swiglu"
    line = {"metric": "e2ttt_decode_tokens_per_s", "value": r.B / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": steps,
            "warmup": max(args.warmup, copies), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"e2ttt_apply, one token per sequence, B={r.B} H={r.H} d={r.d} h={r.h} {kind} {r.io} I/O",
                       "B": r.B, "H": r.H, "d": r.d, "h": r.h, "kind": kind, "io": r.io, "seed": r.seed,
                       "l2": f"steps rotate over {copies} independent state copies ({copies * state_bytes / 1e6:.0f} MB > 126 MB L2)"},
            "e2e": {"value": r.B / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": host_q.numel() * host_q.element_size(),
                    "d2h_bytes_per_step": host_o.numel() * host_o.element_size(), "ms_per_step": ms_e2e},
            "gpu_launches": steps, "clocks": clocks,
            "roofline": {"bound": "hbm", "achieved": nbytes / (ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                         "frac": nbytes / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], "traffic": None, "peak_source": pk["_source"],
                         "kernel": "apply kernel (one launch per step, steps replayed from a CUDA graph)",
                         "bytes_per_launch": nbytes, "ms_per_step_launched_from_python": ms_eager},
            "chunk_update": {"ms": ms_update, "every_tokens": C,
                             "ms_per_token_amortised": ms + ms_update / C,
                             "what": "e2ttt_chunk_fwd over the C accumulated tokens of every sequence (state in, state out)"}}
    print(json.dumps(line))


def run_prepare(args, r):
    """Optional workload (--prepare): one step = e2ttt_prepare_fwd over all token-heads of the configuration (SiLU + L2
    normalisation of q and k, gate parameterisation).  Streaming, HBM-bound: every byte read once, written once."""
    import torch
    from paper_2608_21308_b200 import binding as E

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    iod = torch.float32 if r.io == "f32" else torch.bfloat16
    s4, s3 = (r.B, r.H, r.L, r.d), (r.B, r.H, r.L)
    gen = torch.Generator(device="cpu").manual_seed(r.seed)
    host = {n: torch.randn(s4, generator=gen).to(iod).pin_memory() for n in ("q_raw", "k_raw")}
    host.update({n: (2.0 * torch.randn(s3, generator=gen)).pin_memory() for n in ("a_eta", "a_beta", "a_alpha")})
    t = {n: v.to(dev) for n, v in host.items()}
    q, k = torch.empty_like(t["q_raw"]), torch.empty_like(t["k_raw"])
    eta, beta, gamma = (torch.empty(s3, dtype=torch.float32, device=dev) for _ in range(3))
    hout = [torch.empty_like(host["q_raw"]).pin_memory(), torch.empty_like(host["k_raw"]).pin_memory()] + \
           [torch.empty(s3).pin_memory() for _ in range(3)]
    p = E.make_params(r.B, r.H, r.L, r.d, r.h, r.C, r.kind, E.E2TTT_F32 if r.io == "f32" else E.E2TTT_BF16, 1e-5,
                      E.E2TTT_IMPL_AUTO)
    gp = E.e2ttt_gate_params(0.01, 32.0, 0.1, 1e-12)
    stream = torch.cuda.current_stream()

    def step():
        E.e2ttt_prepare_fwd(p, gp, t["q_raw"], t["k_raw"], t["a_eta"], t["a_beta"], t["a_alpha"], q, k, eta, beta, gamma, stream)

    def step_e2e():
        for n in host:
            t[n].copy_(host[n], non_blocking=True)
        step()
        for a, b in zip(hout, (q, k, eta, beta, gamma)):
            a.copy_(b, non_blocking=True)

    def timed(fn, n, warmup):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    steps = max(args.steps, 20)
    sampler = ClockSampler(0)
    sampler.start()
    ms = timed(step, steps, args.warmup)
    clocks = sampler.stop()
    ms_e2e = timed(step_e2e, max(2, steps // 4), 1)
    # the reverse pass of the same step (training): adjoints of q_raw, k_raw and the gate logits
    dq, dk = torch.randn(s4, generator=gen).to(iod).to(dev), torch.randn(s4, generator=gen).to(iod).to(dev)
    dg = [torch.randn(s3, generator=gen).to(dev) for _ in range(3)]
    dqr, dkr = torch.empty_like(dq), torch.empty_like(dk)
    dlog = [torch.empty(s3, dtype=torch.float32, device=dev) for _ in range(3)]

    def step_bwd():
        E.e2ttt_prepare_bwd(p, gp, t["q_raw"], t["k_raw"], t["a_eta"], t["a_beta"], t["a_alpha"], dq, dk, dg[0], dg[1], dg[2],
                            dqr, dkr, dlog[0], dlog[1], dlog[2], stream)

    ms_bwd = timed(step_bwd, steps, args.warmup)
    pk = peaks()
    rows = r.B * r.H * r.L
    es = 2 if r.io == "bf16" else 4
    nbytes = rows * (4 * r.d * es + 24)
    nbytes_bwd = rows * (6 * r.d * es + 36)
    line = {"metric": "e2ttt_prepare_tokens_per_s", "value": r.B * r.L / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"e2ttt_prepare_fwd B={r.B} H={r.H} L={r.L} d={r.d} {r.io} I/O", "B": r.B, "H": r.H, "L": r.L,
                       "d": r.d, "io": r.io, "seed": r.seed,
                       "l2": f"inputs larger than L2: one step reads and writes {nbytes / 1e6:.0f} MB"},
            "e2e": {"value": r.B * r.L / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": sum(v.numel() * v.element_size() for v in host.values()),
                    "d2h_bytes_per_step": sum(v.numel() * v.element_size() for v in hout), "ms_per_step": ms_e2e},
            "gpu_launches": steps, "clocks": clocks,
            "roofline": {"bound": "hbm", "achieved": nbytes / (ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                         "frac": nbytes / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], "traffic": None, "peak_source": pk["_source"],
                         "kernel": "prepare_fwd_bulk_kernel (one launch per step)", "bytes_per_launch": nbytes},
            "reverse": {"ms_per_step": ms_bwd, "bytes_per_launch": nbytes_bwd,
                        "achieved_gbs": nbytes_bwd / (ms_bwd * 1e-3) / 1e9,
                        "frac_of_hbm_peak": nbytes_bwd / (ms_bwd * 1e-3) / 1e9 / pk["hbm_gbs"],
                        "kernel": "prepare_bwd_bulk_kernel"}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="benchmark configuration index (default: the 1.3B-layer shape)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--backward", action="store_true", help="time forward + backward instead (1 GPU, GELU-MLP configs)")
    ap.add_argument("--ckpt-every", type=int, default=0,
                    help="with --backward: keep the state of every n-th chunk only and recompute n chunks at a time in the "
                         "backward (0: every chunk's state is kept)")
    ap.add_argument("--decode", action="store_true", help="time the decode step instead: e2ttt_apply on one token per sequence (1 GPU)")
    ap.add_argument("--prepare", action="store_true", help="time the token preparation instead (e2ttt_prepare_fwd, 1 GPU)")
    ap.add_argument("--post-norm", action="store_true", help="forward with post-chunk normalisation of the fast weights (e2ttt_chunk_fwd_normed)")
    ap.add_argument("--chunk", type=int, default=0, help="override the chunk size C of the configuration")
    ap.add_argument("--kernel", default="auto", choices=["auto", "fused", "tiled", "simt"],
                    help="kernel family of the forward: auto (the library's choice), fused (tensor-core kernel with the state on "
                         "chip; the library's choice wherever it serves the shape at up to 64 tokens per chunk; chunks of 128, 256, 512 "
                         "tokens must ask for it), tiled / simt (any-shape kernels)")
    ap.add_argument("--gates", default="benchmark", choices=["benchmark", "paper"],
                    help="gate recipe: the benchmark's, or the paper's regime (eta_base 0.01, tau 32, alpha_base 0.1)")
    ap.add_argument("--preroll", type=float, default=1.2,
                    help="seconds of untimed steps under load before the timed ones (clock sampling); 0 = none")
    ap.add_argument("--rank-check", action="store_true",
                    help="no GPU work: every rank joins a gloo group and rank 0 prints the world size (tests the launch path)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as plain `python bench.py --gpus N`: start the N ranks ourselves, one process per GPU
        port = 29500 + (os.getpid() % 2000)
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if args.rank_check:
        import torch.distributed as dist
        dist.init_process_group("gloo")
        import torch
        t = torch.ones(1)
        dist.all_reduce(t)
        if dist.get_rank() == 0:
            print(json.dumps({"rank_check": True, "n_gpus": args.gpus, "world": dist.get_world_size(), "ranks_seen": int(t.item())}))
        dist.destroy_process_group()
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    r = inputs.config(args.config, **({"C": args.chunk} if args.chunk else {}))
    if args.gates == "paper":
        r = inputs.paper_regime(r)
    if args.prepare and args.impl == "ours":
        run_prepare(args, r)
    elif args.decode and args.impl == "ours":
        run_decode(args, r)
    elif args.backward and args.impl == "ours":
        run_fwd_bwd(args, r)
    elif args.impl == "reference":
        run_reference(args, r)
    else:
        run_ours(args, r)


if __name__ == "__main__":
    main()
