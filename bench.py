#!/usr/bin/env python
"""Benchmark of the whitening hot path on a ResNet-shaped layer set.

One step = one pass of the whole path over one batch for every layer of the
set: fw_group_cov_update (Gram + moments), fw_group_cond_reduce (K recursion
steps of P power iterations), fw_group_grad_transform_step (G Qs + SGD).
Metric: whitened layer-updates per second (layers x steps / time).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload resnet20|resnet50|linear|stress|cost_sweep] [--prec fp32|tc]

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
FP32_FFMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12   # SMs x FP32 lanes x 2 flop x max SM clock


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


def make_inputs(spec, layer_ids=None):
    if spec["cfg"] == 4:
        return [synth.cost_sweep_layer(spec["shapes"][0]["B"])]
    out = []
    for i, s in enumerate(spec["shapes"]):
        if layer_ids is not None and i not in layer_ids:
            out.append(None)
            continue
        d = synth.conv_layer_inputs(s["B"], s["HW"], s["C_in"], s["C_out"], s["k"],
                                    synth.layer_seed(spec["cfg"], i), decades=spec["decades"])
        if spec["x_bf16"]:
            d["X"] = synth.to_bf16_grid(d["X"])
        out.append(d)
    return out


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


def oracle_step_time(spec, inputs, steps, layer_ids):
    """Seconds per step of the fp64 oracle over the given layers (as it stands)."""
    from oracle import fw_oracle as O
    layers = {}
    for i in layer_ids:
        d = inputs[i]
        L = O.Layer(d["M"], d["N"], O.Hyper(alpha=spec["alpha"], beta=0.0, gamma=1.0, delta=0.25))
        layers[i] = (L, d["W"].astype(np.float64), d["b"].astype(np.float64))
    t0 = time.perf_counter()
    for _ in range(steps):
        for i in layer_ids:
            L, W, b = layers[i]
            d = inputs[i]
            O.cov_update(L, d["X"])
            O.cond_reduce(L, spec["K"], spec["P"])
            Gt = O.grad_transform(L, d["G"])
            W, b = O.sgd_step(W, b, Gt, d["gb"].astype(np.float64), 0.1)
            layers[i] = (L, W, b)
    return (time.perf_counter() - t0) / steps


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, spec):
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
    # bounded sample: one layer of each distinct shape, scaled to the whole set
    distinct = {}
    for i, s in enumerate(spec["shapes"]):
        distinct.setdefault((s["HW"], s["C_in"], s["C_out"], s["k"]), []).append(i)
    ids = [v[0] for v in distinct.values()]
    if spec["cfg"] == 3:
        ids = [i for i in ids if synth.shape_dims(spec["shapes"][i])[0] * synth.shape_dims(spec["shapes"][i])[1] ** 2 < 3e11]
    inputs = make_inputs(spec, set(ids))
    for _ in range(min(args.warmup, 1)):
        oracle_step_time(spec, inputs, 1, ids)
    steps = max(1, min(args.steps, 3))
    per_layer = {}
    t_total = 0.0
    for i in ids:
        t = oracle_step_time(spec, inputs, steps, [i])
        per_layer[i] = t
    for key, members in distinct.items():
        if members[0] in per_layer:
            t_total += per_layer[members[0]] * len(members)
        else:
            n_layers -= len(members)
    value = n_layers / t_total
    sample = f"one layer of each of {len(ids)} distinct shapes, full rows, {steps} step(s), scaled by multiplicity"
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=steps,
                warmup=min(args.warmup, 1), ms_per_step=t_total * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=spec["name"], layers=n_layers, K=spec["K"], P=spec["P"]),
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


def gram_bound_us(inputs, x_bf16, pk):
    """Sum over layers of max(algorithmic flops / tensor peak, algorithmic bytes / HBM peak): the time the
    Gram pass would take with every layer on its own binding roofline.  Algorithmic flops are the symmetric
    count rows*M*(M+1); the TF32 peak is the measured BF16 peak times the nominal ratio 1/2."""
    tc = pk["bf16_tflops"] * (1.0 if x_bf16 else 0.5) * 1e12
    es = 2 if x_bf16 else 4
    t = 0.0
    for d in inputs:
        flops = float(d["rows"]) * d["M"] * (d["M"] + 1)
        byts = float(d["rows"]) * d["M"] * es + 4.0 * d["M"] ** 2
        t += max(flops / tc, byts / (pk["hbm_gbs"] * 1e9))
    return t * 1e6


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/, for the kernels as they stand; a kernel changed since its capture gets None here.
NCU_TRAFFIC = {
    ("resnet20", "gram"): 660.77e6 + 17.24e6,           # profiles/gram_umma_kernel_resnet20.md
    ("resnet20", "recur_cluster"): 26.25e6 + 0.10e6,    # profiles/recursion_cluster_kernel_resnet20.md
    # cost sweep: Gram launch captured at B = 256 (659.2 MB read + 7.6 MB written); the read part grows with the rows
    ("cost_sweep", "gram_per_256"): 660.76e6,           # profiles/gram_pair_kernel_tf32_cost_sweep_bf16_resnet50.md
    ("cost_sweep", "gram_write"): 8.17e6,
    # stress, M = 2304: captured on 17 layers, proportional to the number of layers
    ("stress2304", "pass_per_layer"): (361.19e6 + 3.95e6) / 17,    # profiles/recursion_pass_kernel_stress_M2304.md
    ("stress2304", "update_per_layer"): (1083.46e6 + 1023.58e6) / 17,  # profiles/recursion_update_kernel_stress_M2304.md
}


def cost_context(spec, inputs, args):
    """Cost sweep only: the cost figures of the paper's complexity analysis, as context.  The paper counts, per
    sample, 2 N M^2 multiply-adds for whitening activations and their gradients directly against N S M^2 / B for
    transforming the weight gradient once per batch (ratio S / (2 B), S the spatial size of a sample); in im2col
    form the same two costs are 4 rows M^2 and 2 N M^2 flop per batch."""
    if spec["cfg"] != 4:
        return {}
    d = inputs[0]
    S = spec["shapes"][0]["HW"] ** 2
    return dict(paper_context=dict(S=S, B=args.B, S_over_2B=S / (2.0 * args.B),
                                   direct_whitening_flop_per_batch=4.0 * d["rows"] * d["M"] ** 2,
                                   gradient_transform_flop_per_batch=2.0 * d["N"] * d["M"] ** 2,
                                   note="direct per-sample whitening is not built; figures from the paper's cost model"))


def run_ours(args, spec):
    import torch
    from paper_2010_01546_b200 import binding as B

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
    dev = torch.device("cuda", local)

    prec = B.FW_PREC_FP32 if args.prec == "fp32" else (B.FW_PREC_BF16 if spec["x_bf16"] else B.FW_PREC_TF32)
    inputs = make_inputs(spec)
    n_layers = len(inputs)
    layers, Xd, Gd, Wd, bd, gbd, Xh, Gh, gbh = [], [], [], [], [], [], [], [], []
    for d in inputs:
        L = B.Layer(d["M"], d["N"], device=dev, alpha=spec["alpha"], beta=0.0, gamma=1.0, delta=0.25,
                    x_dtype=B.FW_BF16 if spec["x_bf16"] else B.FW_F32, prec=prec)
        layers.append(L)
        if spec["x_bf16"]:
            xh = torch.from_numpy(synth.bf16_bits(d["X"]).view(np.int16)).view(torch.bfloat16)
        else:
            xh = torch.from_numpy(d["X"])
        Xh.append(xh.pin_memory()); Gh.append(torch.from_numpy(d["G"]).pin_memory())
        gbh.append(torch.from_numpy(d["gb"]).pin_memory())
        Xd.append(Xh[-1].to(dev)); Gd.append(Gh[-1].to(dev)); gbd.append(gbh[-1].to(dev))
        Wd.append(torch.from_numpy(d["W"]).to(dev)); bd.append(torch.from_numpy(d["b"]).to(dev))
        L.attach_params(Wd[-1], bd[-1])
    hs = [L.handle for L in layers]
    rows = [d["rows"] for d in inputs]
    ldx = [d["M"] for d in inputs]
    K, P, lr = spec["K"], spec["P"], 0.01
    x_bytes = sum(int(x.numel() * x.element_size()) for x in Xd)

    def step(X=Xd, G=Gd, gb=gbd):
        B.fw_group_cov_update(hs, X, rows, ldx)
        B.fw_group_cond_reduce(hs, K, P)
        B.fw_group_grad_transform_step(hs, G, Wd, bd, gb, lr)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    # keep the GPU under the same load until the clock sampler (100 ms period) has something to report
    t_load = time.perf_counter()
    while args.steps >= 10 and time.perf_counter() - t_load < 0.6:
        step()
        torch.cuda.synchronize()
    barrier()
    lc0 = B.fw_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = B.fw_launch_count() - lc0
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(ms, dist, dev)
    value = aggregate_value(n_layers, args.steps, ms, world)

    # per-kernel-class device time over the same number of steps (events around every launch)
    B.fw_profile_begin()
    for _ in range(args.steps):
        step()
    prof = B.fw_profile_end()
    tot = sum(v[0] for v in prof.values()) or 1.0
    shares = {k: round(v[0] / tot, 4) for k, v in prof.items()}
    dom = max(prof, key=lambda k: prof[k][0])
    dom_ms, dom_n = prof[dom]
    pk = peaks()
    m2 = sum(4.0 * d["M"] ** 2 for d in inputs)
    if dom == "gram" and prec == B.FW_PREC_FP32:
        flops = sum(float(d["rows"]) * d["M"] * (d["M"] + 1) for d in inputs)     # SYRK count
        ach = flops / (dom_ms / dom_n * 1e-3) / 1e12
        roof = dict(kernel="gemm_ffma_kernel (Gram, fp32 FFMA)", bound="alu", achieved=ach,
                    peak=FP32_FFMA_PEAK_TFLOPS, unit="TFLOP/s", frac=ach / FP32_FFMA_PEAK_TFLOPS, traffic=None,
                    peak_source="derived: 148 SMs x 128 FP32 lanes x 2 flop x 1.965 GHz")
    elif dom == "gram":
        # the Gram pass of a step is one launch of the single-CTA kernel and/or one of the CTA-pair kernel
        byts = x_bytes + m2
        tc_peak = pk["bf16_tflops"] * (1.0 if spec["x_bf16"] else 0.5)          # TF32 = measured BF16 x 1/2 (nominal)
        flops = sum(float(d["rows"]) * d["M"] * (d["M"] + 1) for d in inputs)     # SYRK count
        step_s = dom_ms / args.steps * 1e-3
        if flops / (tc_peak * 1e12) > byts / (pk["hbm_gbs"] * 1e9):
            ach = flops / step_s / 1e12
            roof = dict(kernel="gram_pair_kernel (Gram pass; flops = rows M (M + 1), the symmetric count)",
                        bound="tensor", achieved=ach, peak=tc_peak, unit="TFLOP/s", frac=ach / tc_peak,
                        traffic=NCU_TRAFFIC.get((args.workload, "gram")),
                        peak_source=pk["source"] + (" bf16" if spec["x_bf16"] else " bf16 x 1/2 (TF32)"))
        else:
            ach = byts / step_s / 1e9
            roof = dict(kernel="gram_umma_kernel + gram_pair_kernel (Gram pass of the set)", bound="hbm",
                        achieved=ach, peak=pk["hbm_gbs"], unit="GB/s", frac=ach / pk["hbm_gbs"],
                        traffic=NCU_TRAFFIC.get((args.workload, "gram")), peak_source=pk["source"])
    else:
        traffic_key = None
        chip_m2 = sum(4.0 * d["M"] ** 2 for d in inputs if d["M"] <= 608)     # layers whose recursion runs on chip
        if dom == "recur_chip":
            # on-chip recursion: one launch runs all K steps; bytes by the multi-pass accounting (P + 11) x 4 M^2
            byts = K * (P + 11) * chip_m2
            name = "recursion_cluster_kernel (K steps on chip; bytes = multi-pass accounting, state is SMEM/L2 resident)"
            traffic_key = (args.workload, "recur_cluster")
        elif dom == "recur_upd":
            byts, name = 6 * (m2 - chip_m2), "recursion_update_kernel"
        elif dom == "recur_mv":
            # one read of the M x M matrix of every streamed layer per matrix-vector launch
            byts, name = m2 - chip_m2, "recursion_pass_kernel (matrix-vector passes of the layers streamed from HBM)"
        else:
            byts, name = m2, dom
        ach = byts / (dom_ms / dom_n * 1e-3) / 1e9
        roof = dict(kernel=name, bound="hbm", achieved=ach, peak=pk["hbm_gbs"], unit="GB/s",
                    frac=ach / pk["hbm_gbs"], traffic=NCU_TRAFFIC.get(traffic_key), peak_source=pk["source"])
        if dom == "recur_chip":
            # the state of these layers sits in shared memory and L2: the passes are latency-bound, so the
            # time per recursion step says more than the bandwidth figure
            roof["us_per_recursion_step"] = dom_ms / dom_n * 1e3 / K
    if "gram" in prof and prec != B.FW_PREC_FP32:
        g_ms, g_n = prof["gram"]
        g_us = g_ms / args.steps * 1e3            # all Gram launches of a step (single-CTA and CTA-pair kernel)
        g_ach = (x_bytes + m2) / (g_us * 1e-6) / 1e9
        bound_us = gram_bound_us(inputs, spec["x_bf16"], pk)
        roof["gram_kernel"] = dict(kernel="gram_umma_kernel + gram_pair_kernel", bound="hbm", achieved=g_ach,
                                   peak=pk["hbm_gbs"], unit="GB/s", frac=g_ach / pk["hbm_gbs"], us_per_step=g_us,
                                   launches_per_step=g_n / args.steps,
                                   traffic=NCU_TRAFFIC.get((args.workload, "gram")),
                                   bound_time_us=bound_us, frac_of_per_layer_bound=bound_us / g_us)
    if spec["cfg"] == 4 and "gram_kernel" in roof:
        # captured at B = 256; the bytes read grow in proportion to the rows, the partials written do not
        tr = NCU_TRAFFIC[("cost_sweep", "gram_per_256")] * args.B / 256.0 + NCU_TRAFFIC[("cost_sweep", "gram_write")]
        roof["gram_kernel"]["traffic"] = tr
        if roof.get("bound") == "tensor":
            roof["traffic"] = tr
    roof["shares"] = shares
    roof["class_us_per_step"] = {k: round(v[0] / args.steps * 1e3, 1) for k, v in prof.items()}
    roof["avg_launch_us"] = dom_ms / dom_n * 1e3

    # end to end: inputs start in pinned host memory every step, the updated weights are read back
    stream = torch.cuda.current_stream()
    Wh = [torch.empty(w.shape, dtype=w.dtype).pin_memory() for w in Wd]
    h2d = x_bytes + sum(int(g.numel() * 4) for g in Gd) + sum(int(g.numel() * 4) for g in gbd)
    d2h = sum(int(w.numel() * 4) for w in Wd)

    def e2e_step():
        for i in range(n_layers):
            Xd[i].copy_(Xh[i], non_blocking=True)
            Gd[i].copy_(Gh[i], non_blocking=True)
            gbd[i].copy_(gbh[i], non_blocking=True)
        step()
        for i in range(n_layers):
            Wh[i].copy_(Wd[i], non_blocking=True)
        stream.synchronize()

    e2e_steps = max(3, min(args.steps, 10))
    e2e_step()
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    ms_e = e0.elapsed_time(e1)
    ms_e = max_over_ranks(ms_e, dist, dev)
    e2e_value = aggregate_value(n_layers, e2e_steps, ms_e, world)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        ids = list(range(n_layers))
        if spec["cfg"] == 3:
            ids = [i for i in ids if inputs[i]["rows"] * inputs[i]["M"] ** 2 < 3e11]
        if spec["cfg"] == 4:
            t_cpu = oracle_cost_sweep_time(spec, inputs[0])
            cpu = dict(value=1.0 / t_cpu, unit=UNIT, cores=cpu_threads(), kind="oracle",
                       sample="moments on the first 12544 rows scaled to %d rows, 2 of %d recursion steps scaled, "
                              "transform in full" % (inputs[0]["rows"], spec["K"]))
        else:
            t_cpu = oracle_step_time(spec, inputs, 1, ids)
            cpu = dict(value=len(ids) / t_cpu, unit=UNIT, cores=cpu_threads(), kind="oracle",
                       sample=f"{len(ids)} of {n_layers} layers, full rows, 1 step of the fp64 numpy oracle")

    if rank == 0:
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps,
                    warmup=max(args.warmup, 3), ms_per_step=ms / args.steps, higher_is_better=True,
                    scaling="weak", vs_baseline=None,
                    dtype="f32" if prec == B.FW_PREC_FP32 else ("bf16" if spec["x_bf16"] else "tf32"),
                    data="synthetic",
                    config=dict(workload=spec["name"], layers=n_layers, K=K, P=P, engine=args.prec,
                                l2="inputs larger than L2 (%.0f MB of X per step)" % (x_bytes / 1e6),
                                multi_gpu="independent replicas, no collective", **cost_context(spec, inputs, args)),
                    clocks=clocks, gpu_launches=int(launches),
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h),
                    roofline=roof, cpu_baseline=cpu)
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------
# recursion stress workload: Phi_x given, many independent layers, recursion only
# ----------------------------------------------------------------------------
def run_stress(args):
    """One step = fw_group_cond_reduce(K = 8, P = 32) over `layers` independent layers with
    Phi_x = U diag(logspace(0, -log10 cond, M)) U^T injected.  Working set 3 x layers x 4 M^2."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    M, nl, K, P = args.M, args.layers, 8, 32
    name = f"recursion_stress_M{M}_x{nl}_cond{args.cond:g}"
    distinct = min(nl, 4)
    phis = [synth.spd_with_spectrum(M, args.cond, synth.layer_seed(5, i), basis="qr" if M <= 512 else "householder")[0]
            .astype(np.float32) for i in range(distinct)]
    if args.impl == "reference":
        if rank != 0:
            return
        from oracle import fw_oracle as O
        L = O.Layer(M, 1, O.Hyper(beta=0.0, gamma=1.0, delta=0.25))
        L.set_phix(phis[0])
        t0 = time.perf_counter()
        O.cond_reduce(L, K, P)
        t = time.perf_counter() - t0
        v = 1.0 / t
        print(json.dumps(dict(impl="reference", metric=METRIC, value=v, unit=UNIT, n_gpus=args.gpus, steps=1, warmup=0,
                              ms_per_step=t * 1e3 * nl, higher_is_better=True, scaling="weak", vs_baseline=None,
                              dtype="f64", data="synthetic", config=dict(workload=name, layers=nl, K=K, P=P),
                              cpu_baseline=dict(value=v, unit=UNIT, cores=cpu_threads(), kind="oracle",
                                                sample="1 layer, K steps of the fp64 numpy oracle"),
                              e2e=dict(value=v, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))
        return
    import torch
    from paper_2010_01546_b200 import binding as B
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist_.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_
    dev = torch.device("cuda", local)
    ph = [torch.from_numpy(p).pin_memory() for p in phis]
    pd = [p.to(dev) for p in ph]
    layers = [B.Layer(M, 16, device=dev, beta=0.0, gamma=1.0, delta=0.25) for _ in range(nl)]
    for i, L in enumerate(layers):
        L.set(B.FW_F_PHIX, pd[i % distinct])
    hs = [L.handle for L in layers]

    def step():
        B.fw_group_cond_reduce(hs, K, P)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    steps = max(1, min(args.steps, 10))
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    lc0 = B.fw_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = B.fw_launch_count() - lc0
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(ms, dist, dev)
    value = aggregate_value(nl, steps, ms, world)
    B.fw_profile_begin()
    step()
    prof = B.fw_profile_end()
    pk = peaks()
    SM = 4.0 * M * M * nl
    clustered = "recur_chip" in prof
    mv_ms, mv_n = prof.get("recur_chip" if clustered else "recur_mv", (0.0, 1))
    up_ms, up_n = prof.get("recur_upd", (0.0, 0))
    if clustered:
        byts = K * (P + 11) * SM
        ach = byts / (mv_ms * 1e-3) / 1e9
        kern = "recursion_cluster_kernel (bytes = multi-pass accounting; state is SMEM/L2 resident)"
    else:
        byts = K * (P + 5) * SM          # P + 4 reads of Phi_y and one of T^T per step
        ach = byts / (mv_ms * 1e-3) / 1e9
        kern = "recursion_pass_kernel (matrix-vector passes)"
    per_layer = NCU_TRAFFIC.get(("stress%d" % M, "pass_per_layer"))
    roof = dict(kernel=kern, bound="hbm", achieved=ach, peak=pk["hbm_gbs"], unit="GB/s", frac=ach / pk["hbm_gbs"],
                traffic=(per_layer * nl if per_layer and not clustered else None), peak_source=pk["source"],
                avg_launch_us=mv_ms / mv_n * 1e3,
                class_us_per_step={k: round(v[0] * 1e3, 1) for k, v in prof.items()})
    if not clustered:
        u_ach = K * 6 * SM / (up_ms * 1e-3) / 1e9
        upl = NCU_TRAFFIC.get(("stress%d" % M, "update_per_layer"))
        roof["update_kernel"] = dict(kernel="recursion_update_kernel", achieved=u_ach, frac=u_ach / pk["hbm_gbs"],
                                     traffic=(upl * nl if upl else None))
        roof["whole_recursion"] = dict(achieved=K * (P + 11) * SM / ((mv_ms + up_ms) * 1e-3) / 1e9,
                                       note="(P + 11) x 4 M^2 bytes per step per layer over matrix-vector + update time")
    # end to end: Phi_x comes from pinned host memory every step, Q is read back
    qh = [torch.empty(M, M, dtype=torch.float32).pin_memory() for _ in range(distinct)]
    stage = [torch.empty(M, M, dtype=torch.float32, device=dev) for _ in range(distinct)]
    def e2e_step():
        for i in range(distinct):
            stage[i].copy_(ph[i], non_blocking=True)
        for i, L in enumerate(layers):
            L.set(B.FW_F_PHIX, stage[i % distinct])
        step()
        for i in range(distinct):
            B.fw_layer_get(hs[i], B.FW_F_Q, stage[i], M * M * 4)
            qh[i].copy_(stage[i], non_blocking=True)
        torch.cuda.synchronize()
    e2e_step()
    barrier()
    e0.record()
    for _ in range(3):
        e2e_step()
    e1.record()
    barrier()
    e2e_value = world * nl * 3 / (e0.elapsed_time(e1) * 1e-3)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import fw_oracle as O
        Lo = O.Layer(M, 1, O.Hyper(beta=0.0, gamma=1.0, delta=0.25))
        Lo.set_phix(phis[0])
        t0 = time.perf_counter()
        O.cond_reduce(Lo, K if M <= 1152 else 2, P)
        t = (time.perf_counter() - t0) * (1 if M <= 1152 else K / 2)
        cpu = dict(value=1.0 / t, unit=UNIT, cores=cpu_threads(), kind="oracle",
                   sample="1 layer of the fp64 numpy oracle" + ("" if M <= 1152 else ", 2 of 8 steps scaled"))
    if rank == 0:
        print(json.dumps(dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=steps,
                              warmup=max(args.warmup, 3), ms_per_step=ms / steps, higher_is_better=True,
                              scaling="weak", vs_baseline=None, dtype="f32", data="synthetic",
                              config=dict(workload=name, layers=nl, K=K, P=P,
                                          l2="working set %.1f GB (3 matrices per layer) larger than L2" % (3 * SM / 1e9),
                                          multi_gpu="independent replicas, no collective"),
                              clocks=clocks, gpu_launches=int(launches),
                              e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=int(distinct * M * M * 4),
                                       d2h_bytes_per_step=int(distinct * M * M * 4)),
                              roofline=roof, cpu_baseline=cpu)))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet20",
                    choices=["resnet20", "resnet50", "linear", "stress", "cost_sweep"])
    ap.add_argument("--B", type=int, default=1024, help="cost_sweep workload: batch size (rows = 196 B)")
    ap.add_argument("--prec", default="tc", choices=["fp32", "tc"],
                    help="tc: tcgen05 tensor cores (TF32 / BF16 inputs, fp32 accumulate); fp32: FFMA engine")
    ap.add_argument("--M", type=int, default=2304, help="stress workload: matrix size")
    ap.add_argument("--layers", type=int, default=64, help="stress workload: independent layers")
    ap.add_argument("--cond", type=float, default=1e4, help="stress workload: condition number of Phi_x")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.workload == "stress":
        run_stress(args)
        return
    spec = workload_spec(args.workload)
    if spec["cfg"] == 4:
        spec["shapes"][0]["B"] = args.B
        spec["name"] += "_B%d" % args.B
        args.steps = min(args.steps, 20)
    if args.impl == "reference":
        run_reference(args, spec)
    else:
        run_ours(args, spec)


if __name__ == "__main__":
    main()
