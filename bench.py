"""Benchmark of the VARCO partitioned-layer path on B200.

One "step" is one epoch of the hot path over the whole graph: every layer of the model forward
(halo gather/compress -> exchange -> decompress -> aggregate -> transform) and backward (transform
gradients -> transposed aggregate -> compress -> return -> ordered add), all partitions, at one
compression ratio.  The metric is partitioned-layer edges per second: stored directed adjacency
entries x layers, divided by the epoch time (forward + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--ratio 1] [--impl ours|reference]

With N > 1 (torchrun, one rank per GPU) every rank runs an independent replica of the workload:
the path is defined on one GPU with no collectives, so the ranks only share the timing barrier.
`--impl reference` times the CPU oracle (a deliberately plain program) on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2406_17611_b200 import synth  # noqa: E402

METRIC = "partitioned_layer_edges_per_s"
UNIT = "edges/s"
SWEEP_RATIOS = [(64, 1), (16, 1), (4, 1), (1, 1)]


def parse_ratio(s):
    if "/" in s:
        a, b = s.split("/")
        return int(a), int(b)
    return int(s), 1


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown," \
        "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown," \
        "clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            tok = [t.strip() for t in line.split(",")]
            if len(tok) < 7:
                continue
            try:
                sm.append(float(tok[0]))
                mx.append(float(tok[1]))
            except ValueError:
                continue
            for nm, v in zip(names, tok[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["sm_max_mhz"] = float(max(mx))
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------------------------------ model on device
class DeviceModel:
    """The workload's tensors resident in HBM and one epoch (all layers fwd + bwd) over them."""

    def __init__(self, wl, device):
        import torch
        from paper_2406_17611_b200 import binding as vb
        self.torch, self.vb, self.wl, self.device = torch, vb, wl, device
        self.dt = torch.bfloat16 if wl.bf16 else torch.float32
        self.es = 2 if wl.bf16 else 4
        self.vec = 16 // self.es
        t0 = time.time()
        self.plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
        self.plan_build_s = time.time() - t0
        self.plan.upload(device)
        self.perm = self.plan.perm()
        self.L = len(wl.widths) - 1
        n = wl.n
        self.ld = [self._ld(f) for f in wl.widths]
        X0 = wl.features()[self.perm]
        self.X0_host = torch.zeros((n, self.ld[0]), dtype=self.dt).pin_memory()
        self.X0_host[:, :wl.widths[0]] = torch.from_numpy(X0).to(self.dt)
        self.acts = [torch.empty((n, self.ld[l]), dtype=self.dt, device=device) for l in range(self.L + 1)]
        self.aggs = [torch.empty((n, self.ld[l]), dtype=self.dt, device=device) for l in range(self.L)]
        self.grads = [torch.empty((n, self.ld[l]), dtype=self.dt, device=device) for l in range(self.L + 1)]
        rng = np.random.default_rng(wl.seed + 7)
        dY = rng.standard_normal((n, wl.widths[-1])).astype(np.float32)
        self.dY_host = torch.zeros((n, self.ld[-1]), dtype=self.dt).pin_memory()
        self.dY_host[:, :wl.widths[-1]] = torch.from_numpy(dY).to(self.dt)
        self.Y_host = torch.empty((n, self.ld[-1]), dtype=self.dt).pin_memory()
        self.W = []
        for l in range(self.L):
            Ws, Wn, b = wl.layer_weights(l)
            dev = lambda a, d: None if a is None else torch.from_numpy(a).to(d).to(device).contiguous()
            f32 = dict(dtype=torch.float32, device=device)
            shape = (wl.widths[l], wl.widths[l + 1])
            self.W.append(dict(Ws=dev(Ws, self.dt), Wn=dev(Wn, self.dt), b=dev(b, torch.float32),
                               dWs=None if Ws is None else torch.empty(shape, **f32),
                               dWn=torch.empty(shape, **f32), db=torch.empty((shape[1],), **f32)))
        self.ws = self.plan.workspace(max(wl.widths[:-1]), max(wl.widths[1:]), vb.BF16 if wl.bf16 else vb.F32, device)
        self.acts[0].copy_(self.X0_host)
        self.grads[self.L].copy_(self.dY_host)
        torch.cuda.synchronize(device)

    def _ld(self, f):
        return (f + self.vec - 1) // self.vec * self.vec

    def _forward(self, ratio, epoch_idx):
        vb, wl = self.vb, self.wl
        total = 0
        for l in range(self.L):
            w = self.W[l]
            _, _, hb = vb.varco_layer_fwd(self.plan, self.acts[l], w["Ws"], w["Wn"], w["b"], l < self.L - 1, ratio,
                                          (wl.seed, epoch_idx, l), self.ws, F_in=wl.widths[l], Y=self.acts[l + 1],
                                          Agg=self.aggs[l])
            total += hb
        return total

    def _backward(self, ratio, epoch_idx):
        vb, wl = self.vb, self.wl
        total = 0
        for l in reversed(range(self.L)):
            w = self.W[l]
            r = vb.varco_layer_bwd(self.plan, self.acts[l], self.acts[l + 1], self.aggs[l], w["Ws"], w["Wn"],
                                   self.grads[l + 1], l < self.L - 1, ratio, (wl.seed, epoch_idx, l), self.ws,
                                   F_in=wl.widths[l], dX=self.grads[l], dW_self=w["dWs"], dW_neigh=w["dWn"],
                                   dbias=w["db"])
            total += r[4]
        return total

    def epoch(self, ratio, epoch_idx):
        """All layers forward then backward.  Returns the halo bytes put on the wire."""
        return self._forward(ratio, epoch_idx) + self._backward(ratio, epoch_idx)

    def epoch_e2e(self, ratio, epoch_idx):
        """The same epoch fed from pinned host memory, results read back to the host, as a pipeline: all copies
        run on a second stream beside the kernels.  The input features of the NEXT step are uploaded into the
        other of two device buffers while this step computes (one upload per step; a step starts once its own
        upload, issued during the step before, has landed); the upstream gradient is only needed by the backward
        pass and the logits are final after the forward pass, so those copies overlap the kernels too."""
        torch = self.torch
        main = torch.cuda.current_stream()
        if not hasattr(self, "_copy_stream"):
            self._copy_stream = torch.cuda.Stream()
            self._x0 = [self.acts[0], torch.empty_like(self.acts[0])]
            self._x0_ready = [None, None]      # upload of the buffer has landed (recorded on the copy stream)
            self._x0_free = [None, None]       # the last step that read the buffer is done (recorded on main)
            self._turn = 0
        side = self._copy_stream
        cur, nxt = self._turn % 2, (self._turn + 1) % 2
        if self._x0_ready[cur] is None:        # very first step: nothing was prefetched
            with torch.cuda.stream(side):
                side.wait_stream(main)
                self._x0[cur].copy_(self.X0_host, non_blocking=True)
                self._x0_ready[cur] = side.record_event()
        with torch.cuda.stream(side):
            if self._x0_free[nxt] is not None:
                side.wait_event(self._x0_free[nxt])
            self._x0[nxt].copy_(self.X0_host, non_blocking=True)        # the next step's input
            self._x0_ready[nxt] = side.record_event()
            side.wait_stream(main)             # the previous backward pass has released the gradient buffer
            self.grads[self.L].copy_(self.dY_host, non_blocking=True)
            dY_ready = side.record_event()
        main.wait_event(self._x0_ready[cur])
        self.acts[0] = self._x0[cur]
        total = self._forward(ratio, epoch_idx)
        fwd_done = main.record_event()
        with torch.cuda.stream(side):
            side.wait_event(fwd_done)
            self.Y_host.copy_(self.acts[self.L], non_blocking=True)
        main.wait_event(dY_ready)
        total += self._backward(ratio, epoch_idx)
        self._x0_free[cur] = main.record_event()
        main.wait_stream(side)
        self._turn += 1
        host = [w["dWn"].cpu() for w in self.W]
        return host

    def e2e_bytes(self):
        h2d = self.X0_host.numel() * self.es + self.dY_host.numel() * self.es
        d2h = self.Y_host.numel() * self.es + sum(w["dWn"].numel() * 4 for w in self.W)
        return h2d, d2h


def measured_traffic(args, stage):
    """DRAM bytes per epoch of one stage from the committed ncu capture, or None when the capture does not
    belong to this workload / ratio or was taken from other kernel sources."""
    path = os.path.join(ROOT, "profiles", "dram_traffic_c3_ratio1.json")
    if args.workload != "c3" or args.scale != 1.0 or parse_ratio(args.ratio) != (1, 1) or args.parts:
        return None
    try:
        from paper_2406_17611_b200.ncu_summary import source_digest
        d = json.load(open(path))
        if d.get("source_sha1") != source_digest():
            return None
        return d["dram_bytes_per_epoch"].get(stage)
    except (OSError, ValueError, KeyError):
        return None


def stage_work(wl, plan, ratio_k):
    """Algorithmic bytes / flops of every stage for ONE epoch (all layers): what the method has to move or
    multiply, every source row counted once."""
    n, nnz, H = wl.n, plan.nnz, plan.H_total
    nnz_f = nnz + (n if wl.conv == "gcn" else 0)
    es = 2 if wl.bf16 else 4
    sage = wl.conv == "sage"
    work = {s: 0.0 for s in ("compress", "decompress", "spmm", "gemm_fwd", "gemm_dx", "gemm_dw", "spmm_t",
                              "compress_bwd", "scatter_add")}
    for l in range(len(wl.widths) - 1):
        F, Fo, k = wl.widths[l], wl.widths[l + 1], ratio_k[l]
        kc = (2 if sage else 1) * F
        work["compress"] += H * (2 * k * es + 4)
        work["decompress"] += H * (k * es + F * es)
        work["spmm"] += nnz_f * 4 + (n + H) * F * es + n * F * es + (n + 1) * 8
        work["spmm_t"] += nnz_f * 4 + n * F * es + (n + H) * F * es + (n + H + 1) * 8
        work["compress_bwd"] += plan_nb(plan) * k * 2 if k < F else 0   # 16-bit kept positions, once per boundary row
        work["scatter_add"] += H * k * es + 2 * plan_nb(plan) * F * es
        work["gemm_fwd"] += 2.0 * n * kc * Fo
        work["gemm_dx"] += 2.0 * n * kc * Fo
        work["gemm_dw"] += 2.0 * n * kc * Fo
    return work


def plan_nb(plan):
    return plan.boundary_rows


# ------------------------------------------------------------------------------------------ oracle legs
class OracleSample:
    """The CPU oracle, as it stands, on one epoch of a scaled-down instance of the workload."""

    def __init__(self, wl_name, sample_scale, threads=None):
        import oracle
        self.orc = oracle.Oracle()
        if threads:
            self.orc.set_threads(threads)
        wl = self.wl = synth.make_workload(wl_name, sample_scale)
        self.g = self.orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
        self.es = 2 if wl.bf16 else 4
        self.L = len(wl.widths) - 1
        self.X = wl.features().astype(np.float64)
        self.dY = np.random.default_rng(wl.seed + 7).standard_normal((wl.n, wl.widths[-1]))
        self.weights = [wl.layer_weights(l) for l in range(self.L)]

    def epoch(self, ratio):
        wl, g, L = self.wl, self.g, self.L
        t0 = time.perf_counter()
        acts = [self.X]
        for l in range(L):
            Ws, Wn, b = self.weights[l]
            Y, _, _ = g.layer_fwd(acts[l], Ws, Wn, b, l < L - 1, ratio, (wl.seed, 0, l), elem_bytes=self.es)
            acts.append(Y)
        grad = self.dY
        for l in reversed(range(L)):
            Ws, Wn, b = self.weights[l]
            grad = g.layer_bwd(acts[l], acts[l + 1], Ws, Wn, grad, l < L - 1, ratio, (wl.seed, 0, l),
                               elem_bytes=self.es)[0]
        dt = time.perf_counter() - t0
        return {"seconds": dt, "edges": wl.nnz * L, "n": wl.n, "nnz": wl.nnz, "threads": self.orc.threads()}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ratio = parse_ratio(args.ratio)
    scale = args.ref_scale
    cores = len(os.sched_getaffinity(0))
    sample_run = OracleSample(args.workload, scale)
    for _ in range(args.warmup):
        sample_run.epoch(ratio)
    times, last = [], None
    for _ in range(args.steps):
        last = sample_run.epoch(ratio)
        times.append(last["seconds"])
    total = sum(times)
    value = last["edges"] * args.steps / total
    sample = "one epoch (all layers fwd+bwd) of the %s generator at scale %g: n=%d, nnz=%d" % (
        args.workload, scale, last["n"], last["nnz"])
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample_scale": scale, "ratio": "%d/%d" % ratio},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["threads"], "kind": "oracle",
                             "sample": sample, "host_cores": cores},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ ours
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2406_17611_b200 import binding as vb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    vb.lib()
    torch.cuda.set_device(local)
    device = "cuda:%d" % local
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ratio = parse_ratio(args.ratio)
    t0 = time.time()
    wl = synth.make_workload(args.workload, args.scale)
    if args.parts:
        wl.part = synth.partition_bfs_ranges(wl.row_ptr, wl.col, args.parts, wl.seed + 1)
        wl.parts = args.parts
        wl.note += " (repartitioned into %d BFS ranges)" % args.parts
    gen_s = time.time() - t0
    model = DeviceModel(wl, device)
    L = model.L
    ks = [vb.varco_kept(wl.widths[l], ratio) for l in range(L)]
    stream_evt = lambda: torch.cuda.Event(enable_timing=True)

    # warm-up
    for w in range(args.warmup):
        model.epoch(ratio, w)
    barrier()

    # timed region: K epochs, per-stage events recorded by the library on the launch stream
    model.plan.profile_enable(True)
    model.plan.profile_reset()
    launches0 = vb.varco_kernel_launches()
    clocks = ClockSampler(local)
    barrier()
    e0, e1 = stream_evt(), stream_evt()
    e0.record()
    halo_bytes = 0
    for s in range(args.steps):
        halo_bytes = model.epoch(ratio, args.warmup + s)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clock_info = clocks.stop()
    launches = vb.varco_kernel_launches() - launches0
    stages = model.plan.profile_read()
    model.plan.profile_enable(False)
    model.plan.profile_reset()
    if world > 1:
        t = torch.tensor([ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    ms_per_step = ms / args.steps
    edges_per_step = wl.nnz * L
    value = world * edges_per_step / (ms_per_step * 1e-3)

    # end to end: inputs from pinned host memory, results back to the host, inside the timed region
    for _ in range(2):
        model.epoch_e2e(ratio, 0)
    barrier()
    e0, e1 = stream_evt(), stream_evt()
    n_e2e = max(3, min(args.steps, 10))
    t_host = time.perf_counter()
    e0.record()
    for s in range(n_e2e):
        model.epoch_e2e(ratio, s)
    e1.record()
    barrier()
    wall_ms = 1e3 * (time.perf_counter() - t_host)
    ms_e2e = max(e0.elapsed_time(e1), 0.0)
    if world > 1:
        t = torch.tensor([ms_e2e], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_e2e = float(t.item())
    h2d, d2h = model.e2e_bytes()
    e2e = {"value": world * edges_per_step / (ms_e2e / n_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / n_e2e, "host_wall_ms_per_step": wall_ms / n_e2e}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # roofline of the dominant stage
    pk = peaks()
    work = stage_work(wl, model.plan, ks)
    per_stage = {}
    for name, (cnt, tot_ms) in stages.items():
        if cnt == 0:
            continue
        entry = {"launches_per_step": cnt / args.steps, "ms_per_step": tot_ms / args.steps,
                 "share": tot_ms / ms if ms > 0 else None}
        if name in work and tot_ms > 0:
            per_s = work[name] / (tot_ms / args.steps * 1e-3)
            if name.startswith("gemm"):
                entry["tflops"] = per_s / 1e12
            else:
                entry["gbs"] = per_s / 1e9
        per_stage[name] = entry
    dom = max((s for s in per_stage if s != "aux"), key=lambda s: per_stage[s]["ms_per_step"])
    d = per_stage[dom]
    if dom.startswith("gemm"):
        peak = pk["bf16_tflops_sustained"] if wl.bf16 else None
        roof = {"kernel": dom, "bound": "tensor" if wl.bf16 else "alu", "achieved": d["tflops"], "peak": peak,
                "unit": "TFLOP/s", "frac": (d["tflops"] / peak) if peak else None, "traffic": None,
                "peak_source": pk["source"] + " (sustained bf16)"}
        if not wl.bf16:
            # fp32 FFMA peak: 148 SMs x 128 lanes x 2 flop x max SM clock
            peak = 148 * 128 * 2 * 1.965e9 / 1e12
            roof.update(peak=peak, frac=d["tflops"] / peak, peak_source="derived: 148 SM x 128 FFMA x 1965 MHz")
    else:
        roof = {"kernel": dom, "bound": "hbm", "achieved": d["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": d["gbs"] / pk["hbm_gbs"], "traffic": None, "peak_source": pk["source"]}

    roof["traffic"] = measured_traffic(args, dom)
    roof["algorithmic"] = work.get(dom)
    roof["per"] = "epoch (all launches of the stage)"
    if dom in ("spmm", "spmm_t") and all(k == f for k, f in zip(ks, wl.widths[:-1])):
        # The algorithmic bytes count every source row once (an unbounded cache).  What a cache of the L2's size
        # can do at best under a simple model: the most used rows of every partition, as many as fit, are read
        # once, every other row once per use (varco_partition_gather_model).
        l2 = int(torch.cuda.get_device_properties(device).L2_cache_size)
        es = 2 if wl.bf16 else 4
        model_bytes = 0.0
        nnz_f = wl.nnz + (wl.n if wl.conv == "gcn" else 0)
        for l in range(L):
            F = wl.widths[l] if dom == "spmm" or 2 * model.ld[l + 1] > wl.widths[l] else wl.widths[l + 1]
            row = model._ld(F) * es
            _, _, rows_read = model.plan.gather_model(l2 // row, transposed=(dom == "spmm_t"))
            out_rows = wl.n if dom == "spmm" else wl.n + model.plan.H_total
            model_bytes += rows_read * row + nnz_f * 8 + out_rows * row
        t_s = d["ms_per_step"] * 1e-3
        roof["cache_model"] = {"l2_bytes": l2, "bytes": model_bytes, "achieved": model_bytes / t_s / 1e9,
                               "frac": model_bytes / t_s / 1e9 / pk["hbm_gbs"],
                               "note": "DRAM bytes if the most used source rows of each partition, L2's size worth, "
                                       "stayed cached and all others were read once per use"}

    # epoch time versus rate
    sweep = {}
    if not args.no_sweep:
        for r in SWEEP_RATIOS:
            model.epoch(r, 0)
            torch.cuda.synchronize()
            a, b = stream_evt(), stream_evt()
            a.record()
            reps = 3
            hb = 0
            for i in range(reps):
                hb = model.epoch(r, i)
            b.record()
            torch.cuda.synchronize()
            sweep["%d/%d" % r] = {"epoch_ms": a.elapsed_time(b) / reps, "halo_bytes_per_epoch": hb}

    # CPU baseline: the oracle as it stands on a bounded sample
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        s = OracleSample(args.workload, args.ref_scale).epoch(ratio)
        cpu = {"value": s["edges"] / s["seconds"], "unit": UNIT, "cores": s["threads"], "kind": "oracle",
               "sample": "one epoch (all layers fwd+bwd) of the %s generator at scale %g: n=%d, nnz=%d, %.1f s"
                         % (args.workload, args.ref_scale, s["n"], s["nnz"], s["seconds"]),
               "host_cores": len(os.sched_getaffinity(0))}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.bf16 else "f32", "data": "synthetic",
            "config": {"workload": "%s: %s; %d-layer %s %s" % (wl.name, wl.note, L, wl.conv,
                                                                 "-".join(str(w) for w in wl.widths)),
                       "n": wl.n, "nnz": wl.nnz, "partitions": wl.parts, "H_total": model.plan.H_total,
                       "cross_entries": model.plan.cross_entries, "ratio": "%d/%d" % ratio, "kept_per_layer": ks,
                       "halo_bytes_per_epoch": halo_bytes, "multi_gpu": "replicas only",
                       "l2": "inputs larger than L2 (every layer streams > 1 GB)" if wl.n * 256 > 2.6e8
                             else "working set near L2 size; no flush"},
            "clocks": clock_info, "e2e": e2e, "gpu_launches": launches, "roofline": roof, "stages": per_stage,
            "epoch_ms_by_ratio": sweep, "cpu_baseline": cpu,
            "setup_s": {"generate": gen_s, "plan_build": model.plan_build_s}}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--ratio", default="1")
    ap.add_argument("--parts", type=int, default=0, help="override the number of partitions (profiling aid)")
    ap.add_argument("--ref-scale", type=float, default=0.01, dest="ref_scale")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
