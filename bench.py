"""Benchmark of the VARCO partitioned-layer path on B200.

One "step" is one epoch of the hot path over the whole graph: every layer of the model forward
(halo gather/compress -> exchange -> decompress -> aggregate -> transform) and backward (transform
gradients -> transposed aggregate -> compress -> return -> ordered add), all partitions, at one
compression ratio.  The metric is partitioned-layer edges per second: stored directed adjacency
entries x layers, divided by the epoch time (forward + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--ratio 1] [--impl ours|reference]
    python bench.py --workload c5 --schedule      the 100-epoch variable schedule of the rate-sweep configuration
    python bench.py --gather-probe                random-row gather rate of the aggregation kernel (L2 and DRAM)

With N > 1 (torchrun, one rank per GPU) every rank runs an independent replica of the workload:
the path is defined on one GPU with no collectives, so the ranks only share the timing barrier.
`--impl reference` times the CPU oracle (a deliberately plain program) on a bounded sample.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
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
SWEEP_RATIOS = [(1, 0), (64, 1), (16, 1), (4, 1), (2, 1), (1, 1)]   # no communication ... full


def parse_ratio(s):
    if s in ("none", "inf"):       # "no communication": nothing is sent
        return 1, 0
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

    def __init__(self, wl, device, share=None):
        """share: another DeviceModel on the same graph and partition whose plan and workspace are reused."""
        import torch
        from paper_2406_17611_b200 import binding as vb
        self.torch, self.vb, self.wl, self.device = torch, vb, wl, device
        self.dt = torch.bfloat16 if wl.bf16 else torch.float32
        self.es = 2 if wl.bf16 else 4
        self.vec = 16 // self.es
        t0 = time.time()
        if share is None:
            self.plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
            self.plan.upload(device)
        else:
            self.plan = share.plan
        self.plan_build_s = time.time() - t0
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
        need = self.plan.workspace_bytes(max(wl.widths[:-1]), max(wl.widths[1:]), vb.BF16 if wl.bf16 else vb.F32)
        if share is not None and share.ws.numel() >= need:
            self.ws = share.ws
        else:
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


def source_digest() -> str:
    """SHA-1 over the CUDA sources: a traffic table is only quoted for the kernels it was taken from."""
    h = hashlib.sha1()
    csrc = os.path.join(ROOT, "paper_2406_17611_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh", ".h", ".cpp")):
            h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()


def measured_traffic(args, stage):
    """DRAM bytes per epoch of one stage from the committed ncu capture, or None when the capture does not
    belong to this workload / ratio or was taken from other kernel sources."""
    path = os.path.join(ROOT, "profiles", "dram_traffic_c3_ratio1.json")
    if args.workload != "c3" or args.scale != 1.0 or parse_ratio(args.ratio) != (1, 1) or args.parts:
        return None
    try:
        d = json.load(open(path))
        if d.get("source_sha1") != source_digest():
            return None
        return d["dram_bytes_per_epoch"].get(stage)
    except (OSError, ValueError, KeyError):
        return None


def narrow_backward(wl, model, l):
    """The backward of layer l aggregates the F_out-wide dZ (and multiplies afterwards) instead of the F_in-wide
    dZ W^T: bf16 layers whose padded output width is at most half the input width."""
    return wl.bf16 and wl.widths[l + 1] <= 256 and 2 * model.ld[l + 1] <= wl.widths[l]


def stage_work(wl, plan, ratio_k, model=None):
    """Algorithmic bytes / flops of every stage for ONE epoch (all layers): what the method has to move or
    multiply, every source row counted once."""
    n, nnz, H, nb = wl.n, plan.nnz, plan.H_total, plan.boundary_rows
    nnz_f = nnz + (n if wl.conv == "gcn" else 0)
    es = 2 if wl.bf16 else 4
    sage = wl.conv == "sage"
    work = {s: 0.0 for s in ("compress", "decompress", "spmm", "gemm_fwd", "gemm_dx", "gemm_dw", "spmm_t",
                              "compress_bwd", "scatter_add")}
    for l in range(len(wl.widths) - 1):
        F, Fo, k = wl.widths[l], wl.widths[l + 1], ratio_k[l]
        kc = (2 if sage else 1) * F
        index = (2 * nb + H) * 4                      # boundary-row list, its slot ranges, the slots
        if k == F:
            # every unique boundary row is read once and written once per destination
            work["compress"] += nb * F * es + H * F * es + index
        elif k > 0:
            # k kept values of every unique boundary row, one copy per destination, plus the 16-bit positions
            work["compress"] += nb * k * es + H * k * es + index + nb * k * 2
            if 8 * k <= F and F <= 384:
                # the receiver keeps (value, position) pairs, not dense rows (4 bytes per bf16 pair, 8 per fp32 pair)
                work["decompress"] += H * (k * es + k * (4 if wl.bf16 else 8)) + nb * k * 2
            else:
                work["decompress"] += H * (k * es + F * es)
            work["compress_bwd"] += nb * k * 2       # 16-bit kept positions, once per boundary row
            if model is not None and narrow_backward(wl, model, l):
                # narrow layer: the slot gradients are compressed in a pass of their own -- from the F_out-wide
                # slot sums (k <= 16: one dot product per kept entry) or from the dense F-wide product
                src = Fo if (k <= 16 and Fo <= 64) else F
                work["compress_bwd"] += H * (src * es + k * es + 4 + k * 2)
        Hl = H if k > 0 else 0                        # no communication: the halo slots do not exist
        work["spmm"] += nnz_f * 4 + (n + Hl) * F * es + n * F * es + (n + 1) * 8
        Fb = Fo if model is not None and narrow_backward(wl, model, l) else F
        work["spmm_t"] += nnz_f * 4 + n * Fb * es + (n + Hl) * Fb * es + (n + Hl + 1) * 8
        if k > 0:
            work["scatter_add"] += H * k * es + 2 * nb * F * es
        work["gemm_fwd"] += 2.0 * n * kc * Fo
        work["gemm_dx"] += 2.0 * n * kc * Fo
        work["gemm_dw"] += 2.0 * n * kc * Fo
    return work


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


def real_graph_row_sample(wl, ratio, rows_per_layer=1500, seconds=12.0):
    """The oracle, as it stands, on the REAL graph of the workload: sampled rows of every distinct layer shape,
    each evaluated from the definitions (forward row and input-gradient row).  Bounded: stops after `seconds`."""
    import oracle
    orc = oracle.Oracle()
    t0 = time.perf_counter()
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    build_s = time.perf_counter() - t0
    L = len(wl.widths) - 1
    deg = np.diff(wl.row_ptr)
    rng = np.random.default_rng(wl.seed + 17)
    shapes, per_layer = {}, []
    budget = seconds / max(1, len({(wl.widths[l], wl.widths[l + 1]) for l in range(L)}))
    for l in range(L):
        F_in, F_out = wl.widths[l], wl.widths[l + 1]
        if (F_in, F_out) in shapes:
            per_layer.append(dict(shapes[(F_in, F_out)], layer=l))
            continue
        X = rng.standard_normal((wl.n, F_in))
        dY = rng.standard_normal((wl.n, F_out))
        Ws, Wn, b = wl.layer_weights(l)
        relu = l < L - 1
        key = (wl.seed, 0, l)
        done_rows, entries, t_f, t_b = 0, 0, 0.0, 0.0
        Y = np.zeros((wl.n, F_out))
        chunk = 100
        while done_rows < rows_per_layer and t_f + t_b < budget:
            rows = rng.integers(0, wl.n, size=chunk).astype(np.int64)
            a = time.perf_counter()
            Yr, _ = g.layer_fwd_rows(rows, X, Ws, Wn, b, relu, ratio, key)
            c = time.perf_counter()
            Y[rows] = Yr
            g.layer_dx_rows(rows, Y, Ws, Wn, dY, relu, ratio, key)
            d = time.perf_counter()
            t_f += c - a
            t_b += d - c
            done_rows += chunk
            entries += int(deg[rows].sum())
        shapes[(F_in, F_out)] = {"F_in": F_in, "F_out": F_out, "k": orc.kept(F_in, ratio), "rows": done_rows,
                                 "entries": entries, "fwd_s": t_f, "dx_s": t_b}
        per_layer.append(dict(shapes[(F_in, F_out)], layer=l))
    # an epoch is every row of every layer: scale each layer's sample to the whole graph
    est_epoch_s = sum(p["fwd_s"] + p["dx_s"] for p in per_layer if p["rows"]) and \
        sum((p["fwd_s"] + p["dx_s"]) * wl.n / p["rows"] for p in per_layer)
    return {"edges_per_s": wl.nnz * L / est_epoch_s if est_epoch_s else None, "threads": orc.threads(),
            "graph_build_s": build_s, "per_layer": per_layer,
            "note": "rows of the real graph evaluated one by one (forward row, input-gradient row; the weight "
                    "gradient, a reduction over all rows, is not part of a row evaluation); epoch estimate = "
                    "sum over layers of sample time x n / rows"}


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


# ------------------------------------------------------------------------------------------ schedule, probes
def run_schedule(model, K=100, a=5, c_max=128, c_min=1):
    """Epochs 0..K-1 of the variable schedule (linear ratio schedule, slope a), one epoch each, forward and
    backward, timed one by one with CUDA events; totals against K epochs of full communication."""
    torch, vb, wl = model.torch, model.vb, model.wl
    L = model.L
    ratios = [vb.varco_schedule_linear(e, K, a, c_max, c_min) for e in range(K)]
    for r in (ratios[0], (1, 1)):
        model.epoch(r, 0)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    bytes_e = []
    ev[0].record()
    for e in range(K):
        bytes_e.append(model.epoch(ratios[e], e))
        ev[e + 1].record()
    torch.cuda.synchronize()
    series = []
    H, es = model.plan.H_total, model.es
    closed_ok = True
    for e in range(K):
        ks = [vb.varco_kept(wl.widths[l], ratios[e]) for l in range(L)]
        closed = 2 * sum(H * k * es for k in ks)          # forward + backward, every layer
        closed_ok &= closed == bytes_e[e]
        series.append({"e": e, "ratio": "%d/%d" % ratios[e], "k": ks, "ms": round(ev[e].elapsed_time(ev[e + 1]), 3),
                       "halo_bytes": bytes_e[e]})
    full = [s for s in series if s["k"] == list(wl.widths[:-1])]
    full_ms = float(np.median([s["ms"] for s in full])) if full else None
    full_bytes = 2 * sum(H * F * es for F in wl.widths[:-1])
    return {"K": K, "slope_a": a, "c_max": c_max, "c_min": c_min, "layers": L,
            "total_ms": sum(s["ms"] for s in series), "total_halo_bytes": sum(bytes_e),
            "full_communication": {"epoch_ms": full_ms, "total_ms": None if full_ms is None else full_ms * K,
                                   "halo_bytes_per_epoch": full_bytes, "total_halo_bytes": full_bytes * K},
            "first_full_epoch": next((s["e"] for s in series if s["k"] == list(wl.widths[:-1])), None),
            "bytes_match_closed_form": bool(closed_ok), "epochs": series}


def gather_probe(device, row_bytes=512, per_out=64, sizes=(131072, 4194304), out_rows=400000):
    """Random-row gather rate of this GPU (varco_probe_gather: sums of randomly indexed table rows, nothing
    else): a table of 64 MB stays in L2, one of 2 GB does not."""
    import torch
    from paper_2406_17611_b200 import binding as vb
    out = {}
    for rows in sizes:
        table = torch.zeros((rows, row_bytes // 2), dtype=torch.bfloat16, device=device)
        index = torch.randint(0, rows, (out_rows, per_out), dtype=torch.int32, device=device)
        res = torch.empty((out_rows, row_bytes // 2), dtype=torch.bfloat16, device=device)
        for _ in range(3):
            vb.varco_probe_gather(table, index, res)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 10
        a.record()
        for _ in range(reps):
            vb.varco_probe_gather(table, index, res)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / reps
        out["L2" if rows * row_bytes <= (96 << 20) else "DRAM"] = {
            "table_MB": rows * row_bytes >> 20, "row_bytes": row_bytes, "gathers": out_rows * per_out, "ms": ms,
            "gathered_TBps": out_rows * per_out * row_bytes / (ms * 1e-3) / 1e12}
        del table, index, res
        torch.cuda.empty_cache()
    return out


def gemm_layers(model, wl, ks, steps, pk, spans):
    """Per-layer figures of the three GEMM stages from the library's own per-call timings (`spans`: the timed
    executions of each stage in enqueue order)."""
    L, n, H = model.L, wl.n, model.plan.H_total
    sage = wl.conv == "sage"
    es = 2 if wl.bf16 else 4
    out = []
    for st, order in (("gemm_fwd", list(range(L))), ("gemm_dx", list(reversed(range(L)))),
                      ("gemm_dw", list(reversed(range(L))))):
        if len(spans[st]) != steps * L:
            continue
        for pos, l in enumerate(order):
            ms = float(np.median([spans[st][s * L + pos] for s in range(steps)]))
            F, Fo = wl.widths[l], wl.widths[l + 1]
            kc = (2 if sage else 1) * F
            flop = 2.0 * n * kc * Fo
            note = None
            if st == "gemm_dx" and narrow_backward(wl, model, l):
                k = ks[l]
                slot_gemm = not (k < F and k <= 16 and Fo <= 64)
                if slot_gemm and k > 0:
                    flop += 2.0 * H * F * Fo
                note = "narrow backward: rows n (concatenated K)%s" % (" + the H halo-slot rows" if slot_gemm else "")
            e = {"stage": st, "layer": l, "shape": "%d x %d x %d" % (n, kc, Fo), "ms": ms, "tflops": flop / ms / 1e9}
            if wl.bf16:
                e["frac_sustained"] = e["tflops"] / pk["bf16_tflops_sustained"]
                e["frac_burst"] = e["tflops"] / pk["bf16_tflops"]
            # the operands every such product has to stream at least once
            byts = n * kc * es + n * Fo * es + (n * kc * es if st == "gemm_dx" else 0)
            e["hbm_frac_of_operand_bytes"] = byts / (ms * 1e-3) / 1e9 / pk["hbm_gbs"]
            e["bound"] = "tensor" if (wl.bf16 and Fo > 64 and F > 64) else "hbm"
            if note:
                e["note"] = note
            out.append(e)
    return out


def run_training(args, device):
    """Accuracy per floats communicated on the SBM configuration (random 8-way split: most neighbours are remote):
    the variable schedule against full communication, fixed ratios 2 and 4 and no communication, the same
    seeded weights and task for every method.  Test accuracy is evaluated at the method's own final ratio."""
    import torch
    from paper_2406_17611_b200 import binding as vb
    from paper_2406_17611_b200.train import Trainer
    wl = synth.make_workload(args.workload if args.workload in ("c2", "c2r") else "c2r", args.scale)
    X, labels, train = synth.planted_task(wl.extra["block"], wl.widths[0], wl.seed + 5)
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv).upload(device)
    perm = plan.perm()
    K, lr = args.train_epochs, args.lr
    X0 = torch.from_numpy(X[perm]).to(device)
    lab = torch.from_numpy(labels[perm]).to(device)
    trn = torch.from_numpy(train[perm]).to(device)
    methods = {"full communication": lambda e: (1, 1), "no communication": lambda e: (1, 0),
               "fixed ratio 2": lambda e: (2, 1), "fixed ratio 4": lambda e: (4, 1),
               "variable (linear, slope 5, 128 -> 1)": lambda e: vb.varco_schedule_linear(e, K, 5, 128, 1)}
    out = {}
    for name, sched in methods.items():
        weights = [list(wl.layer_weights(l)) for l in range(len(wl.widths) - 1)]
        tr = Trainer(plan, wl.widths, weights, wl.bf16, device)
        total, series = 0, []
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for e in range(K):
            loss, hb = tr.step(X0, lab, trn, sched(e), wl.seed, e, lr)
            total += hb
            if (e + 1) % max(1, K // 10) == 0 or e == K - 1:
                acc = tr.accuracy(X0, lab, ~trn, sched(e), wl.seed, K + e)
                series.append({"epoch": e + 1, "floats_communicated": total // 4, "test_accuracy": acc,
                               "train_loss": float(loss.item())})
        torch.cuda.synchronize()
        out[name] = {"final_test_accuracy": series[-1]["test_accuracy"], "floats_communicated": total // 4,
                     "seconds": time.perf_counter() - t0, "series": series}
        del tr
    full = out["full communication"]["floats_communicated"]
    for v in out.values():
        v["floats_vs_full"] = v["floats_communicated"] / full if full else None
    plan.close()
    return {"training": out, "data": "synthetic",
            "config": {"workload": "%s: %s; %s" % (wl.name, wl.note, "-".join(str(w) for w in wl.widths)),
                       "task": "two classes per community, faint community shift in the features (planted_task)",
                       "epochs": K, "lr": lr, "train_share": 0.5}}


def load_workload(args, parts=None, split=None):
    """The named workload, optionally re-cut into `parts` equal partitions (random, or ranges of a BFS order)."""
    parts = parts or args.parts
    split = split or args.split
    if args.workload == "arx":
        return synth.arxiv_shaped(parts or 16, split or "random", args.scale)
    wl = synth.make_workload(args.workload, args.scale)
    if parts:
        if (split or "bfs") == "random":
            wl.part = synth.partition_random_equal(wl.n, parts, wl.seed + 1)
        else:
            wl.part = synth.partition_bfs_ranges(wl.row_ptr, wl.col, parts, wl.seed + 1)
        wl.parts = parts
        wl.note += " (repartitioned into %d %s parts)" % (parts, "random" if split == "random" else "BFS-range")
    return wl


def q_sweep(args, wl0, device, ratio):
    """Epoch time and halo bytes over the number of workers Q in {2, 4, 8, 16}, random and BFS-range splits
    (the sweep over servers of the paper's Section V, on synthetic inputs)."""
    import torch
    rows = []
    for Q in (2, 4, 8, 16):
        for split in ("random", "bfs"):
            wl = load_workload(args, Q, split)
            m = DeviceModel(wl, device)
            for w in range(3):
                m.epoch(ratio, w)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            hb = 0
            for s in range(args.steps):
                hb = m.epoch(ratio, s)
            b.record()
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / args.steps
            rows.append({"Q": Q, "split": split, "epoch_ms": ms, "edges_per_s": wl.nnz * m.L / (ms * 1e-3),
                         "H_total": m.plan.H_total, "cross_share": m.plan.cross_entries / wl.nnz,
                         "halo_bytes_per_epoch": hb})
            m.plan.close()
            del m
            torch.cuda.empty_cache()
    return {"metric": METRIC, "unit": UNIT, "q_sweep": rows, "data": "synthetic",
            "config": {"workload": "%s: %s" % (wl0.name, wl0.note), "ratio": "%d/%d" % ratio, "n": wl0.n,
                       "nnz": wl0.nnz, "steps": args.steps}}


def max_over_ranks(ms, world, device=None):
    """The slowest rank's time: what a multi-rank number is quoted on (all-reduce MAX; identity on one rank)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(units_per_rank, ms_per_step, world):
    """Whole-job throughput of `world` replicas that each process `units_per_rank` per step."""
    return world * units_per_rank / (ms_per_step * 1e-3)


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
    wl = load_workload(args)
    gen_s = time.time() - t0
    if args.q_sweep:
        if rank == 0:
            print(json.dumps(q_sweep(args, wl, device, ratio)), flush=True)
        return
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
    spans_keep = {st: model.plan.profile_spans(st) for st in ("gemm_fwd", "gemm_dx", "gemm_dw")}
    model.plan.profile_enable(False)
    model.plan.profile_reset()
    ms = max_over_ranks(ms, world, device)
    ms_per_step = ms / args.steps
    edges_per_step = wl.nnz * L
    value = aggregate_value(edges_per_step, ms_per_step, world)

    # end to end: inputs from pinned host memory, results back to the host, inside the timed region
    e2e = None
    if not args.no_e2e:
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
        ms_e2e = max_over_ranks(ms_e2e, world, device)
        h2d, d2h = model.e2e_bytes()
        e2e = {"value": aggregate_value(edges_per_step, ms_e2e / n_e2e, world), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / n_e2e, "host_wall_ms_per_step": wall_ms / n_e2e}
        # latency of ONE isolated step, nothing overlapped: upload of the features and the upstream gradient,
        # the epoch, read-back of the logits and every weight gradient, host wall clock around all of it
        lat = []
        for s in range(3):
            torch.cuda.synchronize()
            t_host = time.perf_counter()
            model.acts[0].copy_(model.X0_host, non_blocking=True)
            model.grads[model.L].copy_(model.dY_host, non_blocking=True)
            model.epoch(ratio, s)
            model.Y_host.copy_(model.acts[model.L], non_blocking=True)
            host = [w[k].cpu() for w in model.W for k in ("dWn", "dWs", "db") if w[k] is not None]
            torch.cuda.synchronize()
            lat.append(1e3 * (time.perf_counter() - t_host))
        e2e["isolated_step_ms"] = float(np.median(lat))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # roofline of the dominant stage
    pk = peaks()
    work = stage_work(wl, model.plan, ks, model)
    per_layer_gemm = gemm_layers(model, wl, ks, args.steps, pk, spans_keep)
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
            # fp32 FFMA peak: SMs x 128 lanes x 2 flop x max SM clock, both read from the device
            props = torch.cuda.get_device_properties(device)
            sms = props.multi_processor_count
            mhz = clock_info.get("sm_max_mhz") or getattr(props, "clock_rate", 1965000) / 1000.0
            peak = sms * 128 * 2 * mhz * 1e6 / 1e12
            roof.update(peak=peak, frac=d["tflops"] / peak,
                        peak_source="derived: %d SM x 128 FFMA x %.0f MHz" % (sms, mhz))
    else:
        roof = {"kernel": dom, "bound": "hbm", "achieved": d["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": d["gbs"] / pk["hbm_gbs"], "traffic": None, "peak_source": pk["source"]}

    # the same figure for every memory-bound stage (algorithmic bytes over the stage's time, of the copy peak)
    roof["by_stage"] = {st: {"achieved_GBps": v["gbs"], "frac": v["gbs"] / pk["hbm_gbs"],
                             "traffic": measured_traffic(args, st), "algorithmic": work.get(st)}
                        for st, v in per_stage.items() if "gbs" in v}
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

    # The aggregation stages gather one source row per stored entry, mostly out of L2: their volume over the
    # rate the same kernels reach on an L2-resident table (measured here, one-partition random graph) says how
    # close they run to the L2-to-SM limit, which binds before HBM does on dense neighbourhoods.
    probe = None
    if wl.bf16 and not args.no_probe:
        probe = gather_probe(device)
        l2_rate = probe["L2"]["gathered_TBps"]
        nnz_f = wl.nnz + (wl.n if wl.conv == "gcn" else 0)
        for st in ("spmm", "spmm_t"):
            if st not in per_stage:
                continue
            gathered = 0.0
            for l in range(L):
                F = wl.widths[l + 1] if st == "spmm_t" and narrow_backward(wl, model, l) else wl.widths[l]
                gathered += nnz_f * model._ld(F) * model.es
            t_s = per_stage[st]["ms_per_step"] * 1e-3
            per_stage[st]["l2_gather"] = {"gathered_bytes": gathered, "achieved_TBps": gathered / t_s / 1e12,
                                          "peak_TBps": l2_rate, "frac": gathered / t_s / 1e12 / l2_rate,
                                          "peak_source": "measured in this run: random 512-byte row gathers from a "
                                                         "64 MB table (varco_probe_gather)"}

    # the variable schedule of the rate-sweep configuration (4-layer model on this graph when the workload is c3)
    schedule = None
    if args.schedule or (args.workload == "c3" and args.scale == 1.0 and not args.no_sweep and world == 1):
        sm = model
        if args.workload == "c3":
            wl5 = dataclasses.replace(wl, name="c5", widths=[100, 256, 256, 256, 47])
            sm = DeviceModel(wl5, device, share=model)
        schedule = run_schedule(sm, K=args.schedule_epochs, a=5)
        schedule["model"] = "%d-layer %s %s" % (sm.L, sm.wl.conv, "-".join(str(w) for w in sm.wl.widths))
        if sm is not model:
            del sm

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

    # CPU baseline: the oracle as it stands on bounded samples
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        s = OracleSample(args.workload, args.ref_scale).epoch(ratio)
        cpu = {"value": s["edges"] / s["seconds"], "unit": UNIT, "cores": s["threads"], "kind": "oracle",
               "sample": "one epoch (all layers fwd+bwd) of the %s generator at scale %g: n=%d, nnz=%d, %.1f s"
                         % (args.workload, args.ref_scale, s["n"], s["nnz"], s["seconds"]),
               "host_cores": len(os.sched_getaffinity(0))}
        # the same on one thread, on a quarter of that sample
        s1 = OracleSample(args.workload, args.ref_scale / 4, threads=1).epoch(ratio)
        cpu["single_thread"] = {"value": s1["edges"] / s1["seconds"], "unit": UNIT, "cores": 1,
                                "sample": "one epoch at scale %g: n=%d, nnz=%d, %.1f s"
                                          % (args.ref_scale / 4, s1["n"], s1["nnz"], s1["seconds"])}
        import oracle
        oracle.Oracle().set_threads(len(os.sched_getaffinity(0)))
        if wl.n >= 200000:
            # the real graph of this run: rows sampled per distinct layer shape, evaluated from the definitions
            cpu["real_graph_rows"] = real_graph_row_sample(wl, ratio)

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
            "gemm_layers": per_layer_gemm, "gather_probe": probe, "epoch_ms_by_ratio": sweep,
            "schedule": schedule, "cpu_baseline": cpu,
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
    ap.add_argument("--parts", type=int, default=0, help="override the number of partitions")
    ap.add_argument("--split", default=None, choices=["random", "bfs"], help="how --parts cuts the graph")
    ap.add_argument("--q-sweep", action="store_true", dest="q_sweep",
                    help="epoch time and halo bytes for 2, 4, 8 and 16 partitions, random and BFS-range splits")
    ap.add_argument("--ref-scale", type=float, default=0.01, dest="ref_scale")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-probe", action="store_true", help="skip the gather-rate probe")
    ap.add_argument("--no-e2e", action="store_true", dest="no_e2e",
                    help="skip the end-to-end leg (profiling aid: fewer launches in the process)")
    ap.add_argument("--schedule", action="store_true",
                    help="run the variable schedule (K epochs, slope 5) on this workload and report the series")
    ap.add_argument("--schedule-epochs", type=int, default=100, dest="schedule_epochs")
    ap.add_argument("--train", action="store_true",
                    help="accuracy per floats communicated on the SBM configuration: variable schedule vs baselines")
    ap.add_argument("--train-epochs", type=int, default=100, dest="train_epochs")
    ap.add_argument("--lr", type=float, default=1.0)
    ap.add_argument("--gather-probe", action="store_true", dest="gather_probe",
                    help="only measure the random-row gather rate of the aggregation kernels and exit")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.gather_probe:
        import torch
        torch.cuda.set_device(0)
        print(json.dumps({"gather_probe": gather_probe("cuda:0")}), flush=True)
        return
    if args.train:
        import torch
        torch.cuda.set_device(0)
        print(json.dumps(run_training(args, "cuda:0")), flush=True)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
