#!/usr/bin/env python
"""Benchmark of the whitening hot path on a ResNet-shaped layer set.

One step = one pass of the whole path over one batch for every layer of the
set: fw_group_cov_update (Gram + moments), fw_group_cond_reduce (K recursion
steps of P power iterations), fw_group_grad_transform_step (G Qs + SGD).
Metric: whitened layer-updates per second (layers x steps / time).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload resnet20|resnet50|linear|stress|cost_sweep] [--prec fp32|tc] [--no-legs]

Protocol.  Inputs rotate over two independent batches (so the moments keep
moving and every recursion step still acts: the line counts the timed recursion
steps whose rank update ran).  The state reached after the warm-up is saved and
put back, outside any timed region, before each measurement.  The K timed
steps run back to back between two events (the headline), with an event after
every step (median / min per step); then `reps` single steps are timed one by
one, each from the saved state.  The default run also times short legs of the
other workloads (ResNet-50-shaped set, cost-sweep layer, recursion stress) and
embeds their rooflines under roofline.workloads.

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has
no exchange step, so there is no collective on the data path.
`--impl reference` times the fp64 CPU oracle on the host cores instead.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2010_01546_b200 import synth  # noqa: E402

METRIC = "whitened_layer_updates_per_s"
UNIT = "layer-updates/s"
SM_COUNT, SM_MAX_GHZ = 148, 1.965
FP32_FFMA_PEAK_TFLOPS = SM_COUNT * 128 * 2 * SM_MAX_GHZ * 1e9 / 1e12   # SMs x FP32 lanes x 2 flop x max SM clock
SMEM_PEAK_GBS = SM_COUNT * 128 * SM_MAX_GHZ                              # 128 bytes per clock per SM


def workload_spec(name: str):
    if name == "resnet20":
        return dict(name="resnet20_cifar_b128", shapes=synth.resnet20_shapes(128), cfg=2, K=4, P=16,
                    alpha=0.9, x_bf16=False, decades=0.0)
    if name == "resnet50":
        return dict(name="resnet50_imagenet_b256", shapes=synth.resnet50_shapes(256), cfg=3, K=4, P=16,
                    alpha=0.9, x_bf16=True, decades=1.0)
    if name == "cost_sweep":
        return dict(name="cost_sweep_conv3x3_c256_14x14", shapes=[dict(B=0, HW=14, C_in=256, C_out=256, k=3)],
                    cfg=4, K=8, P=16, alpha=0.9, x_bf16=False, decades=0.0)
    if name == "linear":
        return dict(name="single_linear_m64_n32_b128", shapes=[dict(B=128, HW=1, C_in=64, C_out=32, k=1)],
                    cfg=1, K=8, P=16, alpha=0.9, x_bf16=False, decades=0.0)
    raise SystemExit(f"unknown workload {name}")


def make_inputs(spec, layer_ids=None, batch_index=0):
    """Host (numpy) inputs of one batch, bit-identical to what the parity tests and the oracle see."""
    if spec["cfg"] == 4:
        return [synth.cost_sweep_layer(spec["shapes"][0]["B"])]
    out = []
    for i, s in enumerate(spec["shapes"]):
        if layer_ids is not None and i not in layer_ids:
            out.append(None)
            continue
        d = synth.conv_layer_inputs(s["B"], s["HW"], s["C_in"], s["C_out"], s["k"],
                                    synth.layer_seed(spec["cfg"], i), decades=spec["decades"], batch_index=batch_index)
        if spec["x_bf16"]:
            d["X"] = synth.to_bf16_grid(d["X"])
        out.append(d)
    return out


def make_inputs_device(torch, dev, spec, batch_index=0):
    """Device-drawn inputs of one batch (same recipe, torch's random stream): timing-only legs."""
    if spec["cfg"] == 4:
        return [synth.cost_sweep_layer_device(torch, dev, spec["shapes"][0]["B"], batch_index=batch_index)]
    return [synth.conv_layer_inputs_device(torch, dev, s["B"], s["HW"], s["C_in"], s["C_out"], s["k"],
                                           synth.layer_seed(spec["cfg"], i), decades=spec["decades"],
                                           bf16=spec["x_bf16"], batch_index=batch_index)
            for i, s in enumerate(spec["shapes"])]


# ----------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------
def oracle_cost_sweep_time(spec, d, sample_rows=12544):
    """Seconds per step of the fp64 oracle on the cost-sweep layer: the moments are timed on the first
    sample_rows rows and scaled by rows / sample_rows (their cost is linear in the rows), the recursion on
    two of the K steps and scaled, the transform and SGD step in full."""
    from oracle import fw_oracle as O
    L = O.Layer(d["M"], d["N"], O.Hyper(alpha=spec["alpha"], beta=0.0, gamma=1.0, delta=0.25))
    t0 = time.perf_counter()
    O.cov_update(L, d["X"][:sample_rows])
    t_cov = (time.perf_counter() - t0) * d["rows"] / sample_rows
    t0 = time.perf_counter()
    O.cond_reduce(L, 2, spec["P"])
    t_rec = (time.perf_counter() - t0) * spec["K"] / 2
    t0 = time.perf_counter()
    Gt = O.grad_transform(L, d["G"])
    O.sgd_step(d["W"].astype(np.float64), d["b"].astype(np.float64), Gt, d["gb"].astype(np.float64), 0.1)
    t_gq = time.perf_counter() - t0
    return t_cov + t_rec + t_gq


class OracleSet:
    """The fp64 oracle, as it stands, stepping over a set of layers."""

    def __init__(self, spec, inputs, layer_ids):
        from oracle import fw_oracle as O
        self.O, self.spec, self.ids = O, spec, list(layer_ids)
        self.layers = {}
        for i in self.ids:
            d = inputs[i]
            L = O.Layer(d["M"], d["N"], O.Hyper(alpha=spec["alpha"], beta=0.0, gamma=1.0, delta=0.25))
            self.layers[i] = [L, d["W"].astype(np.float64), d["b"].astype(np.float64)]

    def step(self, inputs):
        O, spec = self.O, self.spec
        for i in self.ids:
            L, W, b = self.layers[i]
            d = inputs[i]
            O.cov_update(L, d["X"])
            O.cond_reduce(L, spec["K"], spec["P"])
            Gt = O.grad_transform(L, d["G"])
            W, b = O.sgd_step(W, b, Gt, d["gb"].astype(np.float64), 0.1)
            self.layers[i] = [L, W, b]


def oracle_step_time(spec, inputs, steps, layer_ids, warmup=0):
    """Seconds per step of the fp64 oracle over the given layers, measured (nothing extrapolated)."""
    o = OracleSet(spec, inputs, layer_ids)
    for _ in range(warmup):
        o.step(inputs)
    t0 = time.perf_counter()
    for _ in range(steps):
        o.step(inputs)
    return (time.perf_counter() - t0) / steps


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, spec):
    """The reference arm: the oracle on the host cores.  Everything in the line is measured: the sample is a
    subset of the layers at full rows, `config.layers` is the number of layers it holds, ms_per_step the
    measured time of one step over them."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if spec["cfg"] == 4:
        d = make_inputs(spec)[0]
        t = oracle_cost_sweep_time(spec, d)
        sample = ("moments on the first 12544 rows scaled to %d rows, 2 of %d recursion steps scaled, transform in full"
                  % (d["rows"], spec["K"]))
        print(json.dumps(dict(impl="reference", metric=METRIC, value=1.0 / t, unit=UNIT, n_gpus=args.gpus, steps=1,
                              warmup=0, ms_per_step=t * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                              dtype="f64", data="synthetic",
                              config=dict(workload=spec["name"], layers=1, K=spec["K"], P=spec["P"]),
                              cpu_baseline=dict(value=1.0 / t, unit=UNIT, cores=cpu_threads(), kind="oracle", sample=sample),
                              e2e=dict(value=1.0 / t, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))
        return
    n_layers = len(spec["shapes"])
    ids = list(range(n_layers))
    if spec["cfg"] == 3:
        # the largest Grams alone take the fp64 oracle minutes: a bounded sample of the set
        ids = [i for i in ids if synth.shape_dims(spec["shapes"][i])[0] * synth.shape_dims(spec["shapes"][i])[1] ** 2 < 3e11]
    inputs = make_inputs(spec, set(ids))
    steps = max(1, min(args.steps, 3))
    warm = min(args.warmup, 1)
    t = oracle_step_time(spec, inputs, steps, ids, warmup=warm)
    value = len(ids) / t
    sample = (f"all {n_layers} layers" if len(ids) == n_layers else f"{len(ids)} of {n_layers} layers (the smaller ones)") \
        + f", full rows, {steps} timed step(s) after {warm} warm-up, every figure measured"
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=steps,
                warmup=warm, ms_per_step=t * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=spec["name"], layers=len(ids), K=spec["K"], P=spec["P"]),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cpu_threads(), kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# ----------------------------------------------------------------------------
# multi-rank helpers (replicas only: no collective on the data path)
# ----------------------------------------------------------------------------
def max_over_ranks(ms, dist, device):
    """Slowest rank's time: the job's time when every rank runs an independent replica."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(units_per_rank, steps, ms, world):
    """Whole-job throughput: units processed by all ranks over the slowest rank's time."""
    return world * units_per_rank * steps / (ms * 1e-3)


# ----------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.idx = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100", "-i", str(self.idx)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for ln in self.f.read().splitlines():
            t = [x.strip() for x in ln.split(",")]
            if len(t) < 9:
                continue
            try:
                sm.append(float(t[1])); mx.append(float(t[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), t[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out = dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/ (not measured in this run: `traffic_source` names the file); a kernel changed since its capture has
# no entry here and reports null.
NCU_TRAFFIC = {
    ("resnet20", "gram"): (660.70e6 + 16.17e6, "profiles/gram_umma_kernel_resnet20.md"),
    ("resnet20", "recur_chip"): (26.71e6 + 0.43e6, "profiles/recursion_cluster_kernel_resnet20.md"),
    ("resnet20", "gq"): (10.70e6, "profiles/gq_pair_kernel_resnet20.md"),
    # three of the six streamed layers were captured (111 MB of Phi_y of 149 MB): scaled by the state bytes
    ("resnet50", "recur_mv"): ((3.4177e9 + 1.3089e9) * 149.2 / 111.5,
                               "profiles/recursion_persistent_kernel_resnet50_subset.md (x 149/111: state bytes)"),
}
# cost-sweep layer: TF32 Gram pass captured at B = 256 (50176 rows): bytes read, bytes written; the reads are
# proportional to the rows
NCU_COST_SWEEP_GRAM_B256 = (661.26e6, 7.90e6, 50176, "profiles/gram_pair_kernel_tf32_cost_sweep_B256.md (reads x rows / 50176)")
# stress workload, one launch per pass: captured on 8 layers of M = 2304 (traffic is proportional to the layers)
NCU_STRESS_PASS_M2304_L8 = (169.97e6 + 3.67e6, "profiles/recursion_pass_kernel_stress_M2304.md (x layers / 8)")


def traffic_of(key):
    v = NCU_TRAFFIC.get(key)
    return (v[0], v[1]) if v else (None, None)


class LayerSet:
    """The layers of a workload on one device, with `nb` resident input batches to rotate over."""

    FIELDS = ("FW_F_MU", "FW_F_PHIX", "FW_F_PHI_DIAG", "FW_F_LAMBDA_BAR", "FW_F_T", "FW_F_Q")

    def __init__(self, B, torch, dev, spec, prec, batches, nhwc=False):
        """batches: list over batches of lists over layers of dicts with device tensors X (or, with nhwc, the
        activation A), G, gb (and W, b in batch 0)."""
        self.B, self.torch, self.dev, self.spec = B, torch, dev, spec
        self.nhwc = nhwc
        self.chunks = int(spec.get("chunks", 1))
        self.K, self.P, self.lr = spec["K"], spec["P"], 0.01
        self.batches = batches
        self.nb = len(batches)
        d0 = batches[0]
        self.n = len(d0)
        self.dims = [(d["rows"], d["M"], d["N"]) for d in d0]
        self.layers = [B.Layer(d["M"], d["N"], device=dev, alpha=spec["alpha"], beta=0.0, gamma=1.0, delta=0.25,
                               x_dtype=B.FW_BF16 if spec["x_bf16"] else B.FW_F32, prec=prec) for d in d0]
        self.W = [d["W"].clone() for d in d0]
        self.b = [d["b"].clone() for d in d0]
        for L, W, b in zip(self.layers, self.W, self.b):
            L.attach_params(W, b)
        self.hs = [L.handle for L in self.layers]
        self.rows = [d["rows"] for d in d0]
        self.ldx = [d["M"] for d in d0]
        self.saved = None
        self.trace = None
        self.on_chip = [bool(B.fw_recursion_on_chip(L.desc)) for L in self.layers]
        if "A" in d0[0]:
            sh = spec["shapes"]
            self.geo = [[s["B"] for s in sh], [s["HW"] for s in sh], [s["HW"] for s in sh], [s["C_in"] for s in sh],
                        [s["k"] for s in sh]]
            self.scr_bytes = [B.fw_nhwc_scratch_bytes(s["B"], s["HW"], s["HW"], s["C_in"], 3) if s["k"] == 3 else 0
                              for s in sh]
            self.scr = [torch.empty(max(nb, 256), dtype=torch.uint8, device=dev) for nb in self.scr_bytes]

    def step(self, i, trace_slot=None, nhwc=None, bt=None):
        B = self.B
        bt = self.batches[i % self.nb] if bt is None else bt
        if self.nhwc if nhwc is None else nhwc:
            B.fw_group_cov_update_nhwc(self.hs, [d["A"] for d in bt], *self.geo, self.scr, self.scr_bytes)
        else:
            # a block larger than the resident buffer is accumulated chunk by chunk (the same rows stand in for
            # every chunk: the timing does not depend on the values)
            for c in range(self.chunks - 1):
                B.fw_group_cov_update(self.hs, [d["X"] for d in bt], self.rows, self.ldx, B.FW_COV_ACCUMULATE)
            B.fw_group_cov_update(self.hs, [d["X"] for d in bt], self.rows, self.ldx)
        tr = None
        if trace_slot is not None and self.trace is not None:
            tr = [t.data_ptr() + trace_slot * self.K * 16 for t in self.trace]
        B.fw_group_cond_reduce(self.hs, self.K, self.P, tr)
        B.fw_group_grad_transform_step(self.hs, [d["G"] for d in bt], self.W, self.b, [d["gb"] for d in bt], self.lr)

    def alloc_trace(self, slots):
        self.trace = [self.torch.zeros(slots * self.K * 4, dtype=self.torch.float32, device=self.dev) for _ in self.layers]

    def active_steps(self, slots):
        """Of the timed recursion steps, how many ran their rank update (a_e != 0, i.e. g_e != 1)."""
        act = tot = 0
        for t in self.trace:
            g = t.view(-1, 4)[: slots * self.K, 1]
            act += int((g != 1.0).sum().item())
            tot += int(g.numel())
        return act, tot

    def save(self):
        B = self.B
        self.saved = [dict((f, L.get(getattr(B, f)).clone()) for f in self.FIELDS) for L in self.layers]
        self.savedW = [w.clone() for w in self.W]
        self.savedb = [b.clone() for b in self.b]

    def restore(self):
        """Puts the saved state back through fw_layer_set (never inside a timed region)."""
        B = self.B
        for L, sv in zip(self.layers, self.saved):
            L.set(B.FW_F_T, sv["FW_F_T"])            # also recomputes Q = T^T T and marks Phi_y stale
            L.set(B.FW_F_Q, sv["FW_F_Q"])
            L.set(B.FW_F_PHIX, sv["FW_F_PHIX"])
            L.set(B.FW_F_LAMBDA_BAR, sv["FW_F_LAMBDA_BAR"])
            L.set(B.FW_F_MU, sv["FW_F_MU"])
            L.set(B.FW_F_PHI_DIAG, sv["FW_F_PHI_DIAG"])
        for w, s in zip(self.W, self.savedW):
            w.copy_(s)
        for b, s in zip(self.b, self.savedb):
            b.copy_(s)


def to_device_batches(torch, dev, spec, host_batches, with_nhwc=False, rows_resident=True):
    """Device copies of the batches: the patch matrix X (unless rows_resident is False), and with with_nhwc the
    NHWC activation A the patches are cut from, each with its pinned host original."""
    out = []
    for bi, hb in enumerate(host_batches):
        lst = []
        for d in hb:
            e = dict(M=d["M"], N=d["N"], rows=d["rows"], Gh=torch.from_numpy(d["G"]).pin_memory(),
                     gbh=torch.from_numpy(d["gb"]).pin_memory())
            if rows_resident:
                if spec["x_bf16"]:
                    x = torch.from_numpy(synth.bf16_bits(d["X"]).view(np.int16)).view(torch.bfloat16)
                else:
                    x = torch.from_numpy(d["X"])
                e["Xh"] = x.pin_memory()
                e["X"] = e["Xh"].to(dev)
            if with_nhwc:
                e["Ah"] = torch.from_numpy(np.ascontiguousarray(d["fm"])).pin_memory()   # B x H x W x C
                e["A"] = e["Ah"].to(dev)
            e["G"] = e["Gh"].to(dev); e["gb"] = e["gbh"].to(dev)
            if bi == 0:
                e["W"] = torch.from_numpy(d["W"]).to(dev); e["b"] = torch.from_numpy(d["b"]).to(dev)
            lst.append(e)
        out.append(lst)
    return out


def measure(ls, steps, warmup, reps, barrier, sampler=None, hold_s=0.0):
    """Warm-up, save the state, then (1) `steps` steps back to back between two events with an event after each
    step, (2) `reps` single steps, each from the saved state, timed one by one, (3) per-class event timing over
    min(steps, 20) steps.  Returns a dict of raw measurements."""
    torch, B = ls.torch, ls.B
    for i in range(max(warmup, 3)):
        ls.step(i)
    barrier()
    ls.save()
    if sampler is not None:
        sampler.start()
    # keep the GPU under the same load (rotating batches) until the clock sampler (100 ms period) has samples
    t_load = time.perf_counter()
    i = 0
    while hold_s > 0 and time.perf_counter() - t_load < hold_s:
        ls.step(i); i += 1
        torch.cuda.synchronize()
    ls.alloc_trace(steps)
    ls.restore()
    barrier()
    lc0 = B.fw_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    barrier()
    ev[0].record()
    for i in range(steps):
        ls.step(i, trace_slot=i)
        ev[i + 1].record()
    barrier()
    total_ms = ev[0].elapsed_time(ev[steps])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    launches = B.fw_launch_count() - lc0
    clocks = sampler.stop() if sampler is not None else None
    act, tot = ls.active_steps(steps)
    # single steps from the saved state
    rep_ms = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for r in range(reps):
        ls.restore()
        torch.cuda.synchronize()
        e0.record()
        ls.step(r)
        e1.record()
        torch.cuda.synchronize()
        rep_ms.append(e0.elapsed_time(e1))
    # per-class device time (events around every launch), evolving steps from the saved state
    psteps = max(1, min(steps, 20))
    ls.restore()
    torch.cuda.synchronize()
    B.fw_profile_begin()
    for i in range(psteps):
        ls.step(i)
    prof = B.fw_profile_end()
    return dict(total_ms=total_ms, per_step=per_step, launches=launches, clocks=clocks, active=act, rec_steps=tot,
                rep_ms=rep_ms, prof=prof, psteps=psteps)


def class_rooflines(ls, m, pk):
    """Per kernel class: device time per step, algorithmic work, the roofline that binds it and the fraction
    reached.  Bounds are per layer: sum over layers of max(flops / tensor peak, bytes / HBM peak)."""
    spec, prof, ps = ls.spec, m["prof"], m["psteps"]
    K, P = ls.K, ls.P
    hbm = pk["hbm_gbs"] * 1e9
    tc_gram = pk["bf16_tflops"] * (1.0 if spec["x_bf16"] else 0.5) * 1e12     # TF32 = measured BF16 x 1/2 (nominal)
    tc_tf32 = pk["bf16_tflops"] * 0.5 * 1e12
    es = 2 if spec["x_bf16"] else 4
    out = {}

    def us(cls):
        return prof[cls][0] / ps * 1e3 if cls in prof else None

    if "gram" in prof:
        flops = sum(float(r) * M * (M + 1) for r, M, N in ls.dims)                 # symmetric count
        # bytes the pass has to read: the patch matrix once, or, from the activation, one k*k-th of that
        kk = [(sh["k"] ** 2 if ls.nhwc else 1) for sh in spec["shapes"]] if spec["cfg"] != 4 else [1]
        in_bytes = [float(r) * M * es / q + 4.0 * M * M for (r, M, N), q in zip(ls.dims, kk)]
        byts = sum(in_bytes)
        bound = sum(max(float(r) * M * (M + 1) / tc_gram, bb / hbm) for (r, M, N), bb in zip(ls.dims, in_bytes))
        t = us("gram") * 1e-6
        out["gram"] = dict(kernel="gram_umma_kernel + gram_pair_kernel" + (" (implicit im2col from the activation)" if ls.nhwc else ""),
                           us_per_step=us("gram"),
                           launches_per_step=prof["gram"][1] / ps, tflops=flops / t / 1e12, gbs=byts / t / 1e9,
                           frac_tensor=flops / t / tc_gram, frac_hbm=byts / t / hbm,
                           bound_time_us=bound * 1e6, frac_of_per_layer_bound=bound / t)
    if "gq" in prof:
        bound = sum(max(2.0 * N * M * M / tc_tf32, (4.0 * M * M + 8.0 * N * M) / hbm) for r, M, N in ls.dims)
        flops = sum(2.0 * N * M * M for r, M, N in ls.dims)
        byts = sum(4.0 * M * M + 8.0 * N * M for r, M, N in ls.dims)
        t = us("gq") * 1e-6
        out["gq"] = dict(kernel="gq_pair_kernel (+ gq_reduce_kernel)", us_per_step=us("gq"), launches_per_step=prof["gq"][1] / ps,
                         tflops=flops / t / 1e12, gbs=byts / t / 1e9, frac_tensor=flops / t / tc_tf32,
                         frac_hbm=byts / t / hbm, bound_time_us=bound * 1e6, frac_of_per_layer_bound=bound / t)
    m2_stream = sum(4.0 * M * M for (r, M, N), oc in zip(ls.dims, ls.on_chip) if not oc)
    m2_chip = sum(4.0 * M * M for (r, M, N), oc in zip(ls.dims, ls.on_chip) if oc)
    if "recur_mv" in prof and m2_stream > 0 and "recur_upd" not in prof:
        # persistent launch: all K steps, passes and rank updates.  Per step P + 3 reads of Phi_y (the row norms
        # come out of the previous update), one of T^T, and the update's 3 reads + 3 writes; + 1 for the first norms
        byts = (K * (P + 10) + 1) * m2_stream
        t = us("recur_mv") * 1e-6
        out["recur_mv"] = dict(kernel="recursion_persistent_kernel (K steps, passes + rank updates; rows partly "
                                      "resident in shared memory, so DRAM traffic is below this accounting)",
                               us_per_step=us("recur_mv"), us_per_recursion_step=us("recur_mv") / K,
                               launches_per_step=prof["recur_mv"][1] / ps, gbs=byts / t / 1e9, frac_hbm=byts / t / hbm)
    elif "recur_mv" in prof and m2_stream > 0:
        byts = K * (P + 5) * m2_stream            # per step: P + 4 reads of Phi_y and one of T^T
        t = us("recur_mv") * 1e-6
        out["recur_mv"] = dict(kernel="recursion_pass_kernel (layers streamed from HBM)", us_per_step=us("recur_mv"),
                               launches_per_step=prof["recur_mv"][1] / ps, gbs=byts / t / 1e9, frac_hbm=byts / t / hbm)
    if "recur_upd" in prof and m2_stream > 0:
        byts = K * 6 * m2_stream
        t = us("recur_upd") * 1e-6
        out["recur_upd"] = dict(kernel="recursion_update_kernel", us_per_step=us("recur_upd"),
                                launches_per_step=prof["recur_upd"][1] / ps, gbs=byts / t / 1e9,
                                frac_hbm=byts / t / hbm,
                                note="counts all K updates; a step whose a_e rounds to 0 leaves early")
    if "recur_chip" in prof and m2_chip > 0:
        # state in distributed shared memory: per recursion step P + 4 slab-times-vector passes out of shared
        # memory and one update pass (read + write); nothing of Phi_y crosses HBM inside a call
        smem_bytes = K * (P + 6) * m2_chip
        t = us("recur_chip") * 1e-6
        out["recur_chip"] = dict(kernel="recursion_cluster_kernel (state on chip, latency-bound chain of passes)",
                                 us_per_step=us("recur_chip"), us_per_recursion_step=us("recur_chip") / K,
                                 smem_gbs=smem_bytes / t / 1e9, frac_smem=smem_bytes / t / 1e9 / SMEM_PEAK_GBS,
                                 layers=sum(ls.on_chip))
    for cls in ("moments", "resync", "pilot", "smooth", "misc"):
        if cls in prof:
            out[cls] = dict(us_per_step=us(cls), launches_per_step=prof[cls][1] / ps)
    return out


def headline_roofline(ls, m, pk, rl, workload):
    """The roofline object of the dominant kernel class of the step."""
    prof = m["prof"]
    dom = max(prof, key=lambda k: prof[k][0])
    c = rl.get(dom, {})
    if dom == "gram":
        tensor_bound = c["frac_tensor"] > c["frac_hbm"]     # the larger fraction names the nearer roofline
        tr, src = traffic_of((workload, "gram"))
        if workload == "cost_sweep":
            rd, wr, rows0, src = NCU_COST_SWEEP_GRAM_B256
            tr = rd * sum(float(r) for r, _, _ in ls.dims) / rows0 + wr
        if tensor_bound:
            peak = pk["bf16_tflops"] * (1.0 if ls.spec["x_bf16"] else 0.5)
            roof = dict(kernel=c["kernel"] + " (flops = rows M (M + 1), the symmetric count)", bound="tensor",
                        achieved=c["tflops"], peak=peak, unit="TFLOP/s", frac=c["tflops"] / peak, traffic=tr,
                        peak_source=pk["source"] + (" bf16" if ls.spec["x_bf16"] else " bf16 x 1/2 (TF32, nominal ratio)"))
        else:
            roof = dict(kernel=c["kernel"] + " (Gram pass of the set; bytes = X once + 4 M^2)", bound="hbm",
                        achieved=c["gbs"], peak=pk["hbm_gbs"], unit="GB/s", frac=c["frac_hbm"], traffic=tr,
                        peak_source=pk["source"])
        roof["traffic_source"] = src
    elif dom == "recur_chip":
        tr, src = traffic_of((workload, "recur_chip"))
        roof = dict(kernel=c["kernel"], bound="smem", achieved=c["smem_gbs"], peak=SMEM_PEAK_GBS, unit="GB/s",
                    frac=c["frac_smem"], traffic=tr, traffic_source=src,
                    peak_source="derived: 148 SMs x 128 B/clk x 1.965 GHz shared-memory bandwidth",
                    note="state on chip: not an HBM figure; the kernel is a chain of dependent passes, "
                         "us_per_recursion_step is the figure to watch",
                    us_per_recursion_step=c["us_per_recursion_step"])
    elif dom in ("recur_mv", "recur_upd"):
        tr, src = traffic_of((workload, dom))
        roof = dict(kernel=c["kernel"], bound="hbm", achieved=c["gbs"], peak=pk["hbm_gbs"], unit="GB/s",
                    frac=c["frac_hbm"], traffic=tr, traffic_source=src, peak_source=pk["source"])
    elif dom == "gq":
        tr, src = traffic_of((workload, "gq"))
        roof = dict(kernel=c["kernel"], bound="hbm", achieved=c["gbs"], peak=pk["hbm_gbs"], unit="GB/s",
                    frac=c["frac_hbm"], traffic=tr, traffic_source=src, peak_source=pk["source"])
    else:
        roof = dict(kernel=dom, bound="hbm", achieved=None, peak=pk["hbm_gbs"], unit="GB/s", frac=None, traffic=None,
                    traffic_source=None, peak_source=pk["source"])
    roof["dominant_class"] = dom
    roof["avg_launch_us"] = prof[dom][0] / prof[dom][1] * 1e3
    tot = sum(v[0] for v in prof.values()) or 1.0
    roof["shares"] = {k: round(v[0] / tot, 4) for k, v in prof.items()}
    roof["classes"] = {k: {kk: (round(vv, 4) if isinstance(vv, float) else vv) for kk, vv in v.items()} for k, v in rl.items()}
    return roof


def fp32_engine_roofline(ls, m):
    prof, ps = m["prof"], m["psteps"]
    flops = sum(float(r) * M * (M + 1) for r, M, N in ls.dims)
    t = prof["gram"][0] / ps * 1e-3
    ach = flops / t / 1e12
    tot = sum(v[0] for v in prof.values()) or 1.0
    return dict(kernel="gemm_ffma_kernel (Gram, fp32 FFMA)", bound="alu", achieved=ach, peak=FP32_FFMA_PEAK_TFLOPS,
                unit="TFLOP/s", frac=ach / FP32_FFMA_PEAK_TFLOPS, traffic=None, traffic_source=None,
                peak_source="derived: 148 SMs x 128 FP32 lanes x 2 flop x 1.965 GHz",
                shares={k: round(v[0] / tot, 4) for k, v in prof.items()},
                class_us_per_step={k: round(v[0] / ps * 1e3, 1) for k, v in prof.items()})


def timing_summary(m, steps):
    ps = sorted(m["per_step"])
    rp = sorted(m["rep_ms"]) if m["rep_ms"] else [float("nan")]
    return dict(per_step_ms_median=statistics.median(ps), per_step_ms_min=ps[0],
                reps=len(m["rep_ms"]), rep_ms_median=statistics.median(rp), rep_ms_min=rp[0],
                note="per_step: the K timed steps back to back, state evolving; rep: single steps, each from the "
                     "state saved after the warm-up (restored with fw_layer_set outside the timed region)",
                recursion_steps_timed=m["rec_steps"], recursion_steps_with_rank_update=m["active"])


def run_leg(B, torch, dev, name, pk, steps=5, reps=5, Bsweep=1024):
    """A short device-resident leg of another workload: its per-class rooflines with its own clock record."""
    spec = workload_spec(name)
    if spec["cfg"] == 4:
        spec["shapes"][0]["B"] = Bsweep
        spec["name"] += "_B%d" % Bsweep
    prec = B.FW_PREC_BF16 if spec["x_bf16"] else B.FW_PREC_TF32
    batches = [make_inputs_device(torch, dev, spec, batch_index=b) for b in range(2)]
    ls = LayerSet(B, torch, dev, spec, prec, batches)
    sampler = ClockSampler(dev.index or 0)

    def barrier():
        torch.cuda.synchronize()

    m = measure(ls, steps, 3, reps, barrier, sampler, hold_s=0.5)
    rl = class_rooflines(ls, m, pk)
    if spec["cfg"] == 4:
        rl["comparator"] = comparator_times(B, torch, ls, reps=3)
    out = dict(workload=spec["name"], layers=ls.n, K=ls.K, P=ls.P, dtype="bf16" if spec["x_bf16"] else "tf32",
               data="synthetic, drawn on the device (same recipe, torch's random stream)",
               ms_per_step=m["total_ms"] / steps, steps=steps, clocks=m["clocks"], timing=timing_summary(m, steps),
               classes={k: {kk: (round(vv, 4) if isinstance(vv, float) else vv) for kk, vv in v.items()} for k, v in rl.items()})
    del ls, batches
    torch.cuda.empty_cache()
    return out


def evd_leg(B, torch, ls, roof, reps=3):
    """The direct construction beside the recursive one on the same covariances (Sec. 5: O(M^3) against O(M^2)):
    fw_group_evd_whiten over the layers of the set, timed with CUDA events; the state is restored afterwards."""
    scr = [torch.empty(B.fw_evd_scratch_bytes(M), dtype=torch.uint8, device=ls.dev) for _, M, _ in ls.dims]
    nb = [int(t.numel()) for t in scr]
    ls.restore()
    B.fw_group_evd_whiten(ls.hs, scr, nb, 0.0)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    for _ in range(reps):
        e0.record()
        B.fw_group_evd_whiten(ls.hs, scr, nb, 0.0)
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    ls.restore()
    torch.cuda.synchronize()
    rec_us = roof.get("classes", {}).get("recur_chip", {}).get("us_per_step")
    ms = statistics.median(ts)
    flops = sum(12.0 * M ** 3 for _, M, _ in ls.dims)            # per sweep: 3 dot products + 2 x 2 row rotations per pair
    return dict(kernel="jacobi_kernel + evd_finish_kernel + vdv_kernel (fw_group_evd_whiten, fp64)", layers=ls.n,
                ms_per_call=ms, ms_min=min(ts), fp64_flops_per_sweep=flops,
                recursion_us_per_call=rec_us, ratio_to_recursion=(ms * 1e3 / rec_us) if rec_us else None,
                note="one decomposition of every layer's Phi_x against the K recursion steps of a call; the rotation "
                     "kernel is bound by its M - 1 grid barriers per sweep, not by arithmetic")


def stress_measure(B, torch, dev, M, nl, cond, K, P, steps, warmup, barrier, sampler=None):
    """Recursion only: fw_group_cond_reduce(K, P) over nl independent layers with Phi_x injected.  Every timed
    step starts from the injected covariance and T = I (re-injected outside the timed region), so all K steps
    act."""
    distinct = min(nl, 4)
    phis = [synth.spd_with_spectrum(M, cond, synth.layer_seed(5, i), basis="qr" if M <= 512 else "householder")[0]
            .astype(np.float32) for i in range(distinct)]
    ph = [torch.from_numpy(p).pin_memory() for p in phis]
    pd = [p.to(dev) for p in ph]
    layers = [B.Layer(M, 16, device=dev, beta=0.0, gamma=1.0, delta=0.25) for _ in range(nl)]
    hs = [L.handle for L in layers]
    traces = [torch.zeros(K * 4, device=dev) for _ in layers]

    def reset():
        for i, L in enumerate(layers):
            L.reset()
            L.set(B.FW_F_PHIX, pd[i % distinct])

    def step():
        B.fw_group_cond_reduce(hs, K, P, traces)

    reset()
    for _ in range(max(warmup, 3)):
        step()
    barrier()
    if sampler is not None:
        sampler.start()
    lc0 = B.fw_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    per = []
    for _ in range(steps):
        reset()
        B.fw_group_cond_reduce(hs, 0, P)          # the Phi_y refresh after the injection is not part of the step
        barrier()
        e0.record()
        step()
        e1.record()
        barrier()
        per.append(e0.elapsed_time(e1))
    launches = B.fw_launch_count() - lc0
    clocks = sampler.stop() if sampler is not None else None
    act = sum(int((t.view(K, 4)[:, 1] != 1.0).sum().item()) for t in traces)
    reset()
    B.fw_group_cond_reduce(hs, 0, P)
    torch.cuda.synchronize()
    B.fw_profile_begin()
    step()
    prof = B.fw_profile_end()
    return dict(per=per, launches=launches, clocks=clocks, prof=prof, active=act, rec_steps=K * nl, layers=layers,
                hs=hs, ph=ph, phis=phis, distinct=distinct, step=step, reset=reset)


def stress_rooflines(B, m, M, nl, K, P, pk):
    prof = m["prof"]
    SM = 4.0 * M * M * nl
    hbm = pk["hbm_gbs"]
    out = {}
    if "recur_chip" in prof:
        t = prof["recur_chip"][0] * 1e-3
        smem_bytes = K * (P + 6) * SM
        out["recur_chip"] = dict(kernel="recursion_cluster_kernel (state on chip, latency-bound chain of passes)",
                                 us_per_step=t * 1e6, us_per_recursion_step=t * 1e6 / K,
                                 smem_gbs=smem_bytes / t / 1e9, frac_smem=smem_bytes / t / 1e9 / SMEM_PEAK_GBS)
    if "recur_mv" in prof and "recur_upd" not in prof:
        t = prof["recur_mv"][0] * 1e-3
        byts = (K * (P + 10) + 1) * SM
        out["recur_mv"] = dict(kernel="recursion_persistent_kernel (K steps in one launch: P + 3 reads of Phi_y, one of "
                                      "T^T and the 3 + 3 matrix passes of the rank update per step)",
                               us_per_step=t * 1e6, us_per_recursion_step=t * 1e6 / K, launches=prof["recur_mv"][1],
                               gbs=byts / t / 1e9, frac_hbm=byts / t / 1e9 / hbm)
    elif "recur_mv" in prof:
        t = prof["recur_mv"][0] * 1e-3
        byts = K * (P + 5) * SM
        out["recur_mv"] = dict(kernel="recursion_pass_kernel (matrix-vector passes, streamed from HBM)",
                               us_per_step=t * 1e6, launches=prof["recur_mv"][1], gbs=byts / t / 1e9,
                               frac_hbm=byts / t / 1e9 / hbm, avg_launch_us=t * 1e6 / prof["recur_mv"][1])
    if "recur_upd" in prof:
        t = prof["recur_upd"][0] * 1e-3
        byts = K * 6 * SM
        out["recur_upd"] = dict(kernel="recursion_update_kernel", us_per_step=t * 1e6, launches=prof["recur_upd"][1],
                                gbs=byts / t / 1e9, frac_hbm=byts / t / 1e9 / hbm)
    if "recur_mv" in prof and "recur_upd" in prof:
        t = (prof["recur_mv"][0] + prof["recur_upd"][0]) * 1e-3
        out["whole_recursion"] = dict(gbs=K * (P + 11) * SM / t / 1e9, frac_hbm=K * (P + 11) * SM / t / 1e9 / hbm,
                                      note="(P + 11) x 4 M^2 bytes per step per layer over matrix-vector + update time")
    return {k: {kk: (round(vv, 4) if isinstance(vv, float) else vv) for kk, vv in v.items()} for k, v in out.items()}


def run_stress_leg(B, torch, dev, M, nl, pk, cond=1e4, K=8, P=32, steps=3):
    sampler = ClockSampler(dev.index or 0)
    m = stress_measure(B, torch, dev, M, nl, cond, K, P, steps, 3, torch.cuda.synchronize, sampler)
    out = dict(workload=f"recursion_stress_M{M}_x{nl}_cond{cond:g}", layers=nl, K=K, P=P, dtype="f32",
               ms_per_step=statistics.median(m["per"]), ms_per_step_min=min(m["per"]), steps=steps, clocks=m["clocks"],
               recursion_steps_timed=m["rec_steps"], recursion_steps_with_rank_update=m["active"],
               classes=stress_rooflines(B, m, M, nl, K, P, pk))
    del m
    torch.cuda.empty_cache()
    return out


def comparator_times(B, torch, ls, reps=5):
    """The cost comparison of Sec. 5 measured: the direct method whitens every sample forward (Eq. 11) and sends
    its gradient back through the transform (Eq. 14), two rows x M x M products per batch; the gradient method
    multiplies the N x M weight gradient by Q once (Eq. 29).  Device times of both on the resident layer."""
    L, d = ls.layers[0], ls.batches[0][0]
    rows, M, N = d["rows"], d["M"], d["N"]
    X = d["X"]
    Y = torch.empty_like(X); dY = torch.randn_like(X); dX = torch.empty_like(X)
    Gt = torch.empty_like(d["G"])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn):
        fn(); torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            e0.record(); fn(); e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return statistics.median(ts)

    t_fwd = timed(lambda: B.fw_whiten_forward(L.handle, X, rows, Y)) * ls.chunks
    t_bwd = timed(lambda: B.fw_whiten_backward(L.handle, dY, rows, dX)) * ls.chunks
    t_gq = timed(lambda: B.fw_grad_transform(L.handle, d["G"], Gt))
    del Y, dY, dX
    torch.cuda.empty_cache()
    rows_all = rows * ls.chunks
    return dict(explicit_forward_us=t_fwd, explicit_backward_us=t_bwd, gradient_transform_us=t_gq,
                measured_time_ratio=(t_fwd + t_bwd) / t_gq,
                flop_ratio_im2col=4.0 * rows_all * M * M / (2.0 * N * M * M),
                explicit_tflops=4.0 * rows_all * M * M / ((t_fwd + t_bwd) * 1e-6) / 1e12,
                gradient_tflops=2.0 * N * M * M / (t_gq * 1e-6) / 1e12,
                note="explicit = fw_whiten_forward + fw_whiten_backward over the batch's rows (TF32 tensor cores); "
                     "gradient = fw_grad_transform; the gradient product is a few tens of microseconds, "
                     "bound by reading Q once and by launch latency, so the time ratio falls short of the flop ratio")


def cost_context(spec, inputs, args):
    """Cost sweep only: the cost figures of the paper's complexity analysis, as context.  The paper counts, per
    sample, 2 N M^2 multiply-adds for whitening activations and their gradients directly against N S M^2 / B for
    transforming the weight gradient once per batch (ratio S / (2 B), S the spatial size of a sample); in im2col
    form the same two costs are 4 rows M^2 and 2 N M^2 flop per batch."""
    if spec["cfg"] != 4:
        return {}
    d = inputs[0]
    S = spec["shapes"][0]["HW"] ** 2
    ch = int(spec.get("chunks", 1))
    return dict(paper_context=dict(S=S, B=args.B, S_over_2B=S / (2.0 * args.B), two_B_over_S=2.0 * args.B / S,
                                   direct_whitening_flop_per_batch=4.0 * d["rows"] * ch * d["M"] ** 2,
                                   gradient_transform_flop_per_batch=2.0 * d["N"] * d["M"] ** 2,
                                   note="the paper's saving factor S / (2 B) counts S output positions per sample; in "
                                        "patch-row form the flop ratio direct / gradient is 2 rows / N"))


def setup_dist(torch):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist_.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_
    return world, rank, local, dist, torch.device("cuda", local)


def run_ours(args, spec):
    import torch
    from paper_2010_01546_b200 import binding as B

    world, rank, local, dist, dev = setup_dist(torch)
    prec = B.FW_PREC_FP32 if args.prec == "fp32" else (B.FW_PREC_BF16 if spec["x_bf16"] else B.FW_PREC_TF32)
    # Layer sets of 3 x 3 fp32 convolutions can also be fed the NHWC activations the patches are cut from (implicit
    # im2col): that is what a framework holds, so the end-to-end leg uses it; the device-resident leg takes the
    # patch matrices (--input rows, the default) or the activations (--input nhwc).
    can_nhwc = (prec == B.FW_PREC_TF32 and spec["cfg"] == 2)
    nhwc = can_nhwc and args.input == "nhwc"
    # the activations of a step are smaller than L2 (126 MB): with them as the resident input, four batches are in
    # rotation, so that a batch has been evicted by the time it comes round again
    nb = (4 if nhwc else 2) if spec["cfg"] != 4 or spec["shapes"][0]["B"] <= 1024 else 1
    host_batches = [make_inputs(spec, batch_index=b) for b in range(nb)] if spec["cfg"] != 4 else \
        [make_inputs(spec)] * 1
    batches = to_device_batches(torch, dev, spec, host_batches, with_nhwc=can_nhwc, rows_resident=not nhwc)
    if spec["cfg"] == 4 and nb == 2:
        # second batch of the single large layer: drawn on the device (the host generator takes minutes at this size)
        d2 = synth.cost_sweep_layer_device(torch, dev, spec["shapes"][0]["B"], batch_index=1)
        e = dict(batches[0][0]); e.update(X=d2["X"], G=d2["G"], gb=d2["gb"]); e.pop("W", None); e.pop("b", None)
        batches.append([e])
    ls = LayerSet(B, torch, dev, spec, prec, batches, nhwc)
    n_layers = ls.n
    xkey = "A" if nhwc else "X"
    x_bytes = sum(int(d[xkey].numel() * d[xkey].element_size()) for d in batches[0])

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    m = measure(ls, args.steps, args.warmup, args.reps, barrier, sampler, hold_s=0.6 if args.steps >= 10 else 0.0)
    ms = max_over_ranks(m["total_ms"], dist, dev)
    value = aggregate_value(n_layers, args.steps, ms, world)
    pk = peaks()
    if prec == B.FW_PREC_FP32:
        roof = fp32_engine_roofline(ls, m)
    else:
        roof = headline_roofline(ls, m, pk, class_rooflines(ls, m, pk), args.workload)
    roof["timing"] = timing_summary(m, args.steps)

    # end to end: the step's inputs start in pinned host memory every step, the updated weights are read back
    stream = torch.cuda.current_stream()
    Wh = [torch.empty(w.shape, dtype=w.dtype).pin_memory() for w in ls.W]
    ekey = "A" if can_nhwc else "X"          # what the host hands over: the activations where the path takes them
    hb = [bt for bt in batches if (ekey + "h") in bt[0]]
    h2d = sum(int(d[ekey].numel() * d[ekey].element_size()) for d in batches[0]) \
        + sum(int(d["G"].numel() * 4 + d["gb"].numel() * 4) for d in batches[0])
    d2h = sum(int(w.numel() * 4) for w in ls.W)

    # A step's inputs travel as one pinned buffer and one copy (the layers' tensors are views into it), on a copy
    # stream that runs one step ahead of the compute stream: the copy of step i + 1 overlaps the kernels of step i,
    # as an input pipeline would.  Every step's inputs are copied and every step's weights are read back inside the
    # timed region.
    def flat_batch(bt):
        items, off = [], 0
        for d in bt:
            for key in (ekey, "G", "gb"):
                src = d[key + "h"]
                nbytes = int(src.numel() * src.element_size())
                items.append((key, src, off, nbytes))
                off += (nbytes + 255) // 256 * 256
        host = torch.empty(off, dtype=torch.uint8).pin_memory()
        devb = torch.empty(off, dtype=torch.uint8, device=dev)
        views, it = [], iter(items)
        for d in bt:
            v = {}
            for _ in range(3):
                key, src, o, nbytes = next(it)
                host[o:o + nbytes].view(src.dtype).view(src.shape).copy_(src)
                v[key] = devb[o:o + nbytes].view(src.dtype).view(src.shape)
            views.append(v)
        return dict(host=host, dev=devb, views=views)

    flats = [flat_batch(bt) for bt in hb[:2]]
    nf = len(flats)
    copy_stream = torch.cuda.Stream(device=dev)
    ev_copied = [torch.cuda.Event() for _ in range(nf)]
    ev_free = [torch.cuda.Event() for _ in range(nf)]

    def e2e_prefetch(i):
        f = flats[i % nf]
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(ev_free[i % nf])          # the step that last read this buffer has finished
            f["dev"].copy_(f["host"], non_blocking=True)
            ev_copied[i % nf].record(copy_stream)

    def e2e_step(i, last):
        if not last and nf > 1:
            e2e_prefetch(i + 1)
        stream.wait_event(ev_copied[i % nf])
        ls.step(i, nhwc=can_nhwc, bt=flats[i % nf]["views"])
        ev_free[i % nf].record(stream)
        if not last and nf == 1:
            e2e_prefetch(i + 1)                              # a single buffer: the copy follows the step that read it
        for w, wh in zip(ls.W, Wh):
            wh.copy_(w, non_blocking=True)

    e2e_steps = max(3, min(args.steps, 10))
    ls.restore()
    for f_ev in ev_free:
        f_ev.record(stream)
    e2e_prefetch(0)
    e2e_step(0, True)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    e2e_prefetch(0)
    for i in range(e2e_steps):
        e2e_step(i, i == e2e_steps - 1)
    e1.record()
    barrier()
    ms_e = max_over_ranks(e0.elapsed_time(e1), dist, dev)
    e2e_value = aggregate_value(n_layers, e2e_steps, ms_e, world)

    legs = None
    n_batches = len(batches)
    evd = None
    if rank == 0 and world == 1 and args.legs and args.workload == "resnet20" and prec != B.FW_PREC_FP32:
        evd = evd_leg(B, torch, ls, roof)
        del ls, batches, hb
        torch.cuda.empty_cache()
        legs = {}
        legs["resnet50"] = run_leg(B, torch, dev, "resnet50", pk)
        legs["cost_sweep_B1024"] = run_leg(B, torch, dev, "cost_sweep", pk, Bsweep=1024)
        legs["stress_M2304"] = run_stress_leg(B, torch, dev, 2304, 64, pk)
        legs["stress_M1152"] = run_stress_leg(B, torch, dev, 1152, 64, pk)
        legs["evd_whitening_resnet20"] = evd
        roof["workloads"] = legs

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        ids = list(range(n_layers))
        if spec["cfg"] == 3:
            ids = [i for i in ids if host_batches[0][i]["rows"] * host_batches[0][i]["M"] ** 2 < 3e11]
        if spec["cfg"] == 4:
            t_cpu = oracle_cost_sweep_time(spec, host_batches[0][0])
            cpu = dict(value=1.0 / t_cpu, unit=UNIT, cores=cpu_threads(), kind="oracle",
                       sample="moments on the first 12544 rows scaled to %d rows, 2 of %d recursion steps scaled, "
                              "transform in full" % (host_batches[0][0]["rows"], spec["K"]))
        else:
            t_cpu = oracle_step_time(spec, host_batches[0], 1, ids)
            cpu = dict(value=len(ids) / t_cpu, unit=UNIT, cores=cpu_threads(), kind="oracle",
                       sample=f"{len(ids)} of {n_layers} layers, full rows, 1 step of the fp64 numpy oracle")

    if spec["cfg"] == 4 and rank == 0 and prec != B.FW_PREC_FP32:
        roof["comparator"] = comparator_times(B, torch, ls)
    if rank == 0:
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps,
                    warmup=max(args.warmup, 3), ms_per_step=ms / args.steps, higher_is_better=True,
                    scaling="weak", vs_baseline=None,
                    dtype="f32" if prec == B.FW_PREC_FP32 else ("bf16" if spec["x_bf16"] else "tf32"),
                    data="synthetic",
                    config=dict(workload=spec["name"], layers=n_layers, K=spec["K"], P=spec["P"], engine=args.prec,
                                input=("NHWC activations (implicit im2col)" if nhwc else "patch matrices (materialised im2col)"),
                                l2="%.0f MB of input per step, %d batches in rotation (%.0f MB, L2 is 126 MB)"
                                   % (x_bytes / 1e6, n_batches, x_bytes * n_batches / 1e6),
                                multi_gpu="independent replicas, no collective", **cost_context(spec, host_batches[0], args)),
                    clocks=m["clocks"], gpu_launches=int(m["launches"]),
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                             input=("NHWC activations from pinned host memory, fw_group_cov_update_nhwc (implicit im2col)"
                                    if can_nhwc else "patch matrices from pinned host memory"),
                             pipeline="one host-to-device copy per step (all layers' inputs in one pinned buffer) on a "
                                      "copy stream one step ahead of the compute stream; weights read back every step"),
                    roofline=roof, cpu_baseline=cpu)
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------
# recursion stress workload: Phi_x given, many independent layers, recursion only
# ----------------------------------------------------------------------------
def run_stress(args):
    """One step = fw_group_cond_reduce(K, P = 32) over `layers` independent layers with
    Phi_x = U diag(logspace(0, -log10 cond, M)) U^T injected.  Working set 3 x layers x 4 M^2.
    With --cond-report the condition number of Phi_y after every step is printed next to the oracle's
    (two layers, untimed)."""
    rank = int(os.environ.get("RANK", "0"))
    M, nl, K, P = args.M, args.layers, args.K, 32
    name = f"recursion_stress_M{M}_x{nl}_cond{args.cond:g}_K{K}"
    if args.impl == "reference":
        if rank != 0:
            return
        from oracle import fw_oracle as O
        phi = synth.spd_with_spectrum(M, args.cond, synth.layer_seed(5, 0), basis="qr" if M <= 512 else "householder")[0]
        L = O.Layer(M, 1, O.Hyper(beta=0.0, gamma=1.0, delta=0.25))
        L.set_phix(phi.astype(np.float32))
        t0 = time.perf_counter()
        O.cond_reduce(L, K, P)
        t = time.perf_counter() - t0
        v = 1.0 / t
        print(json.dumps(dict(impl="reference", metric=METRIC, value=v, unit=UNIT, n_gpus=args.gpus, steps=1, warmup=0,
                              ms_per_step=t * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                              dtype="f64", data="synthetic", config=dict(workload=name, layers=1, K=K, P=P),
                              cpu_baseline=dict(value=v, unit=UNIT, cores=cpu_threads(), kind="oracle",
                                                sample="1 layer, K steps of the fp64 numpy oracle, measured"),
                              e2e=dict(value=v, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))
        return
    import torch
    from paper_2010_01546_b200 import binding as B
    world, rank, local, dist, dev = setup_dist(torch)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    steps = max(1, min(args.steps, 10))
    sampler = ClockSampler(local) if rank == 0 else None
    m = stress_measure(B, torch, dev, M, nl, args.cond, K, P, steps, args.warmup, barrier, sampler)
    ms = max_over_ranks(statistics.median(m["per"]), dist, dev)
    value = aggregate_value(nl, 1, ms, world)
    pk = peaks()
    cl = stress_rooflines(B, m, M, nl, K, P, pk)
    if "recur_mv" in cl:
        c = cl["recur_mv"]
        tr, src = None, None
        if M == 2304 and "recursion_pass_kernel" in c["kernel"]:
            tr, src = NCU_STRESS_PASS_M2304_L8[0] * nl / 8.0, NCU_STRESS_PASS_M2304_L8[1]
        roof = dict(kernel=c["kernel"], bound="hbm", achieved=c["gbs"], peak=pk["hbm_gbs"], unit="GB/s",
                    frac=c["frac_hbm"], traffic=tr, traffic_source=src, peak_source=pk["source"])
    else:
        c = cl["recur_chip"]
        roof = dict(kernel=c["kernel"], bound="smem", achieved=c["smem_gbs"], peak=SMEM_PEAK_GBS, unit="GB/s",
                    frac=c["frac_smem"], traffic=None, traffic_source=None,
                    peak_source="derived: 148 SMs x 128 B/clk x 1.965 GHz shared-memory bandwidth")
    roof["classes"] = cl
    # end to end: Phi_x comes from pinned host memory every step, Q is read back
    layers, hs, ph, distinct = m["layers"], m["hs"], m["ph"], m["distinct"]
    qh = [torch.empty(M, M, dtype=torch.float32).pin_memory() for _ in range(distinct)]
    stage = [torch.empty(M, M, dtype=torch.float32, device=dev) for _ in range(distinct)]

    def e2e_step():
        for i in range(distinct):
            stage[i].copy_(ph[i], non_blocking=True)
        for i, L in enumerate(layers):
            L.set(B.FW_F_PHIX, stage[i % distinct])
        m["step"]()
        for i in range(distinct):
            B.fw_layer_get(hs[i], B.FW_F_Q, stage[i], M * M * 4)
            qh[i].copy_(stage[i], non_blocking=True)
        torch.cuda.synchronize()

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        e2e_step()
    e1.record()
    barrier()
    e2e_value = world * nl * 3 / (e0.elapsed_time(e1) * 1e-3)
    cond_report = None
    if rank == 0 and args.cond_report:
        cond_report = stress_cond_report(B, torch, dev, M, args.cond, K, P)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import fw_oracle as O
        Lo = O.Layer(M, 1, O.Hyper(beta=0.0, gamma=1.0, delta=0.25))
        Lo.set_phix(m["phis"][0])
        ks = K if M <= 1152 else min(K, 2)
        t0 = time.perf_counter()
        O.cond_reduce(Lo, ks, P)
        t = (time.perf_counter() - t0) * K / ks
        cpu = dict(value=1.0 / t, unit=UNIT, cores=cpu_threads(), kind="oracle",
                   sample="1 layer of the fp64 numpy oracle" + ("" if ks == K else f", {ks} of {K} steps scaled"))
    if rank == 0:
        SM = 4.0 * M * M * nl
        print(json.dumps(dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=steps,
                              warmup=max(args.warmup, 3), ms_per_step=ms, higher_is_better=True,
                              scaling="weak", vs_baseline=None, dtype="f32", data="synthetic",
                              config=dict(workload=name, layers=nl, K=K, P=P,
                                          l2="working set %.1f GB (3 matrices per layer) larger than L2" % (3 * SM / 1e9),
                                          timing="median of single steps, each from the injected covariance and T = I",
                                          recursion_steps_timed=m["rec_steps"],
                                          recursion_steps_with_rank_update=m["active"],
                                          multi_gpu="independent replicas, no collective"),
                              clocks=m["clocks"], gpu_launches=int(m["launches"]),
                              e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=int(distinct * M * M * 4),
                                       d2h_bytes_per_step=int(distinct * M * M * 4)),
                              roofline=roof, cpu_baseline=cpu, condition_numbers=cond_report)))
    if dist is not None:
        dist.destroy_process_group()


def stress_cond_report(B, torch, dev, M, cond, K, P, n_layers=2):
    """Condition number of Phi_y after every recursion step, device against oracle (untimed; the oracle's
    eigenvalue routine evaluates both states in fp64)."""
    from oracle import fw_oracle as O
    rep = []
    for li in range(n_layers):
        phi = synth.spd_with_spectrum(M, cond, synth.layer_seed(5, li), basis="qr" if M <= 512 else "householder")[0]
        phi32 = phi.astype(np.float32); phi32 = np.triu(phi32) + np.triu(phi32, 1).T
        L = B.Layer(M, 4, device=dev, beta=0.0, gamma=1.0, delta=0.25)
        L.set(B.FW_F_PHIX, torch.from_numpy(phi32).to(dev))
        Lo = O.Layer(M, 4, O.Hyper(beta=0.0, gamma=1.0, delta=0.25))
        Lo.set_phix(phi32)
        dev_c, ora_c = [O.condition_number(phi32.astype(np.float64))], [O.condition_number(Lo.Phix)]
        for _ in range(K):
            L.cond_reduce(1, P)
            O.cond_reduce(Lo, 1, P)
            dev_c.append(O.condition_number(L.get(B.FW_F_PHIY).cpu().numpy().astype(np.float64)))
            ora_c.append(O.condition_number(Lo.phiy()))
        rep.append(dict(layer=li, device=[float("%.6g" % c) for c in dev_c], oracle=[float("%.6g" % c) for c in ora_c]))
    return rep


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--reps", type=int, default=20, help="single steps timed one by one from the saved state")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet20",
                    choices=["resnet20", "resnet50", "linear", "stress", "cost_sweep"])
    ap.add_argument("--B", type=int, default=1024, help="cost_sweep workload: batch size (rows = 196 B)")
    ap.add_argument("--prec", default="tc", choices=["fp32", "tc"],
                    help="tc: tcgen05 tensor cores (TF32 / BF16 inputs, fp32 accumulate); fp32: FFMA engine")
    ap.add_argument("--M", type=int, default=2304, help="stress workload: matrix size")
    ap.add_argument("--layers", type=int, default=64, help="stress workload: independent layers")
    ap.add_argument("--cond", type=float, default=1e4, help="stress workload: condition number of Phi_x")
    ap.add_argument("--K", type=int, default=8, help="stress workload: recursion steps per call")
    ap.add_argument("--cond-report", action="store_true",
                    help="stress workload: condition number after each step, device against oracle (two layers)")
    ap.add_argument("--input", default="rows", choices=["nhwc", "rows"],
                    help="resident input of the device-timed leg of the ResNet-20-shaped set: materialised patch rows "
                         "(default) or the NHWC activations (implicit im2col); the end-to-end leg feeds the activations")
    ap.add_argument("--layer-subset", default="",
                    help="comma-separated layer indices of the workload to keep (a small case of the same kernels, "
                         "for profiler captures); the workload name gains a suffix")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", dest="legs", action="store_false",
                    help="default workload only: skip the short legs of the other workloads")
    args = ap.parse_args()
    if args.workload == "stress":
        run_stress(args)
        return
    spec = workload_spec(args.workload)
    if spec["cfg"] == 4:
        spec["name"] += "_B%d" % args.B
        # past B = 4096 the block is accumulated over chunks of 4096 samples (7.4 GB of patch rows resident)
        spec["chunks"] = max(1, args.B // 4096)
        spec["shapes"][0]["B"] = args.B // spec["chunks"]
        args.steps = min(args.steps, 20)
    if args.layer_subset:
        keep = [int(t) for t in args.layer_subset.split(",")]
        spec["shapes"] = [spec["shapes"][i] for i in keep]
        spec["name"] += "_layers_" + "_".join(str(i) for i in keep)
    if args.impl == "reference":
        run_reference(args, spec)
    else:
        run_ours(args, spec)


if __name__ == "__main__":
    main()
