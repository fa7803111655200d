#!/usr/bin/env python
"""Decode-throughput benchmark of the hybrid SQ/VQ projection stack.

One step = one decode pass over every projection of every layer of a seeded synthetic
RWKV-6-shaped stack (time-mix R/K/V/G/O, channel-mix K/R/V, the five token-shift mixes fused),
issued as one persistent launch (rwkvq_step_run).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W]
        headline: the 14B-class stack at decode batch 16, every layer's weights distinct, drawn and
        quantized on the device; the same line carries a "configs" map with the 1.6B-class stack at
        batch 1 and the 7B-class stack at batch 1 and 8, a prefill leg (one 7B-class layer, M = 2048),
        a quantizer leg and a proxy leg
  python bench.py --workload c2_1p6b|c3_7b|c4_14b [--batch B] ...   # one stack only
  python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs an independent
replica of the same stack (the path has no exchange step); the value is the tokens all ranks
processed divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one step_kernel launch divided by its
# algorithmic bytes, from an ncu capture of the 1.6B-class stack (about 0.55 GB per launch; the larger
# stacks are beyond the size a capture should hold on the device).  The packed weights are read once
# whatever the stack, so the traffic of a larger stack is this ratio times its algorithmic bytes.
# None = no capture of the kernel as it stands.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.0131    # 538.6 MB of DRAM traffic for 531.6 MB algorithmic

HEADLINE = ("c4_14b", 16)
CONFIGS = (("c2_1p6b", 1), ("c3_7b", 1), ("c3_7b", 8))

METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=["c2_1p6b", "c3_7b", "c4_14b"],
                    help="time this stack only (default: the 14B-class headline plus the configs map)")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--distinct-layers", type=int, default=0,
                    help="draw and quantize weights for this many layers and reuse their values, in "
                         "separate device buffers, for the others (0 = every layer distinct)")
    ap.add_argument("--force-method", default=None, choices=[None, "sq", "vq"],
                    help="pack every matrix with one format instead of the proxy's choice")
    ap.add_argument("--mode", default="step", choices=["step", "ops"],
                    help="step = one persistent launch per step; ops = one rwkvq_gemv launch per product")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true", help="skip the prefill leg (one 7B-class layer, M = 2048)")
    ap.add_argument("--stage-group", type=int, default=0,
                    help="diagnostic: put this many consecutive products into one stage instead of the layer's own "
                         "four dependent stages (0 = the real dependencies); a large value removes every grid barrier "
                         "and shows the streaming rate of the kernel alone")
    ap.add_argument("--quantizer", default="device", choices=["host", "device"],
                    help="where the stack's weights are quantized and packed: rwkvq_pack or rwkvq_quantize_dev")
    ap.add_argument("--weights", default=None, choices=["host", "device"],
                    help="where the synthetic weights are drawn: the numpy generators of the inputs module, or a seeded "
                         "generator on the device (default: device with --quantizer device, else host)")
    ap.add_argument("--no-configs", action="store_true", help="skip the configs map (the other stacks)")
    ap.add_argument("--no-proxy", action="store_true", help="skip the proxy leg")
    ap.add_argument("--no-block", action="store_true", help="skip the chained-block leg")
    ap.add_argument("--no-quantize", action="store_true", help="skip the device-quantizer leg (one 7B-class layer)")
    return ap.parse_args(argv)


def workload_name(spec_name, batch):
    from paper_2505_03803_b200 import inputs
    sp = inputs.STACKS[spec_name]
    return (f"{spec_name}: RWKV-6-shaped stack d={sp['d']} h={sp['h']} L={sp['layers']}, 8 projections + 5 fused "
            f"token-shift mixes per layer, hybrid SQ(3-bit g128)/VQ(2-D, {sp['entries']} entries) by proxy, "
            f"decode batch {batch}")


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for (t, r) in self.rows if (t0 is None or t >= t0) and (t1 is None or t <= t1 + 0.2)]
        if not rows:
            rows = [r for (_, r) in self.rows]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# rank aggregation (host logic; also exercised on CPU with the gloo backend)
# ---------------------------------------------------------------------------------------------
def aggregate_over_ranks(local_ms: float, local_units: float, dist=None):
    """(max over ranks of the elapsed milliseconds, sum over ranks of the units processed)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms), float(local_units)
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------------
# CPU oracle leg
# ---------------------------------------------------------------------------------------------
def oracle_sample(spec_name: str, batch: int, rows_fraction: float = 1.0):
    """Seeded logical codes and activations of ONE layer of the workload (random valid codes; the
    matrix that the seeded coin makes heavy-tailed is VQ-coded, the others SQ), optionally cut to
    the first `rows_fraction` of each matrix's rows (whole 256-row tiles)."""
    from paper_2505_03803_b200 import inputs
    sp = inputs.STACKS[spec_name]
    bits = 6 if sp["entries"] == 64 else 8
    items = []
    for (name, oc, ic, has_mu, stage) in inputs.layer_shapes(sp["d"], sp["h"]):
        seed = inputs.seed_of(spec_name, 0, name)
        roc = max(256, int(oc * rows_fraction) // 256 * 256)
        if inputs.weight_kind(seed) == "gauss":
            codes, method = inputs.random_sq_codes(seed, roc, ic), "sq"
        else:
            codes, method = inputs.random_vq_codes(seed, roc, ic, bits), "vq"
        mu = inputs.random_mu_codes(seed + 1, ic, bits) if has_mu else None
        if has_mu:
            x, xp = inputs.gen_activation_pair(seed + 2, batch, ic, sp["outliers"])
            xp = xp.astype(np.float16)
        else:
            x, xp = inputs.gen_activation(seed + 2, batch, ic, sp["outliers"]), None
        items.append(dict(method=method, codes=codes, mu=mu, x=x.astype(np.float16), xp=xp, oc=roc, ic=ic))
    return items, sp


def oracle_step(items):
    """The oracle's dequantize-and-multiply over the sample, as it stands (fp64)."""
    from oracle import rwkvq_oracle as orc
    out = []
    for it in items:
        c = it["codes"]
        w_hat = orc.sq_decode(c["q"], c["scale"], c["zero"]) if it["method"] == "sq" else orc.vq_decode(c["codebook"], c["q"])
        x = it["x"].astype(np.float64)
        if it["mu"] is not None:
            x = orc.token_shift(x, it["xp"].astype(np.float64), orc.mu_decode(it["mu"]["codebook"], it["mu"]["q"]))
        out.append(orc.gemv(w_hat, x))
    return out


def cpu_threads():
    try:
        import threadpoolctl
        n = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(spec_name, batch, budget_s=12.0, rows_fraction=1.0, steps=None, warmup=0):
    """Times the oracle on one layer (or a row slice of it) and scales to the whole stack."""
    items, sp = oracle_sample(spec_name, batch, rows_fraction)
    sample_weights = sum(it["oc"] * it["ic"] for it in items)
    from paper_2505_03803_b200 import inputs
    total_weights = sum(oc * ic for (_, oc, ic, _, _) in inputs.layer_shapes(sp["d"], sp["h"])) * sp["layers"]
    for _ in range(warmup):
        oracle_step(items)
    times = []
    t_start = time.time()
    while True:
        t0 = time.perf_counter()
        oracle_step(items)
        times.append(time.perf_counter() - t0)
        if steps is not None:
            if len(times) >= steps:
                break
        elif time.time() - t_start >= budget_s or len(times) >= 50:
            break
    per_step = sum(times) / len(times)
    full_step_s = per_step * total_weights / sample_weights
    return dict(value=batch / full_step_s, per_sample_s=per_step, n=len(times), sample_weights=sample_weights,
                total_weights=total_weights, full_step_s=full_step_s)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2505_03803_b200 import inputs
    wl = args.workload or HEADLINE[0]
    sp = inputs.STACKS[wl]
    batch = args.batch or (HEADLINE[1] if args.workload is None else sp["batches"][0])
    K = args.steps if args.steps is not None else 5
    W = args.warmup if args.warmup is not None else 1
    # size the per-step sample from a probe so that the whole run stays near two minutes
    probe = time_oracle(wl, batch, steps=1, rows_fraction=0.125)
    full_layer_s = probe["per_sample_s"] * 8.0
    frac = min(1.0, max(0.125, 120.0 / max(1e-9, full_layer_s * (K + W))))
    frac = max(0.125, int(frac * 8) / 8.0)
    r = time_oracle(wl, batch, steps=K, warmup=W, rows_fraction=frac)
    cores = cpu_threads()
    sample = (f"per step: the oracle's decode + token shift + fp64 product over the first {frac:g} of the rows of "
              f"each of the 8 matrices of one layer ({r['sample_weights']} of {r['total_weights']} weights), "
              f"time scaled to the whole stack by weight count")
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus, "steps": K,
        "warmup": W, "ms_per_step": r["full_step_s"] * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(wl, batch), "batch": batch},
        "cpu_baseline": {"value": r["value"], "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ---------------------------------------------------------------------------------------------
# prefill leg: one 7B-class layer, M = 2048 tokens, through rwkvq_gemm_prefill
# ---------------------------------------------------------------------------------------------
def measured_bf16_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


def _prefill_layer(formats, M):
    """Device buffers of the eight projections of one 7B-class layer, matrix i packed as formats[i]
    ("sq" or "vq"): random valid logical codes (the time does not depend on the code values)."""
    import torch
    from paper_2505_03803_b200 import binding as B
    from paper_2505_03803_b200 import inputs
    sp = inputs.STACKS["c3_7b"]
    mats = []
    for fmt, (name, oc, ic, has_mu, stage) in zip(formats, inputs.layer_shapes(sp["d"], sp["h"])):
        seed = inputs.seed_of("c5_prefill", name)
        if fmt == "sq":
            blob = B.rwkvq_pack(None, oc, ic, B.RWKVQ_SQ, 3, codes=inputs.random_sq_codes(seed, oc, ic))
        else:
            blob = B.rwkvq_pack(None, oc, ic, B.RWKVQ_VQ, 6, codes=inputs.random_vq_codes(seed, oc, ic, 6))
        mu = B.rwkvq_pack(None, 1, ic, B.RWKVQ_VQ, 6, codes=inputs.random_mu_codes(seed + 1, ic)) if has_mu else None
        x = inputs.gen_activation(seed + 2, M, ic, sp["outliers"])
        X = torch.from_numpy(inputs.to_bf16_bits(x).view(np.int16)).cuda().view(torch.bfloat16)
        Y = torch.empty((M, oc), dtype=torch.float32, device="cuda")
        ws = torch.empty(B.rwkvq_prefill_workspace_bytes(blob.desc, M, has_mu), dtype=torch.uint8, device="cuda")
        mats.append((blob.desc, blob.to_device(), mu.desc if mu else None, mu.to_device() if mu else None, X, Y, ws, oc, ic))
    return mats


def _time_prefill_layer(mats, M, reps):
    import torch
    from paper_2505_03803_b200 import binding as B

    # the eight products are independent here (each has its own input), so the layer is one group
    ops, _keep = B.make_prefill_ops([dict(desc=d, W=W, mu_desc=md, mu=m, X=X, Y=Y, workspace=ws)
                                     for (d, W, md, m, X, Y, ws, oc, ic) in mats])

    def layer():
        B.rwkvq_gemm_prefill_grouped(ops, M)
    for _ in range(3):
        layer()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        layer()
    e1.record()
    torch.cuda.synchronize()
    if B.rwkvq_device_status() != 0:
        raise SystemExit("bench.py: a device-side wait timed out in the prefill leg")
    ms = e0.elapsed_time(e1) / reps
    flops = sum(2.0 * M * oc * ic for (*_r, oc, ic) in mats)
    return ms, flops, flops / (ms * 1e-3) / 1e12


def prefill_formats():
    """Formats of the timed hybrid layer: per matrix the seeded coin of the decode stacks (heavy-tailed
    -> VQ-64, Gaussian -> SQ), under the first salt that gives the layer both formats."""
    from paper_2505_03803_b200 import inputs
    sp = inputs.STACKS["c3_7b"]
    names = [name for (name, *_r) in inputs.layer_shapes(sp["d"], sp["h"])]
    for salt in range(64):
        f = ["sq" if inputs.weight_kind(inputs.seed_of("c5_prefill", salt, n)) == "gauss" else "vq" for n in names]
        if 0 < f.count("sq") < len(f):
            return f
    raise SystemExit("bench.py: no seeded hybrid layer found")


def prefill_leg(reps: int = 10, M: int = 2048):
    """All eight projections of one 7B-class layer (d = 4096, h = 14336) over M tokens with the
    token-shift mix on R, K, V, G and cm_k: the hybrid layer (SQ and VQ-64 matrices by the seeded coin),
    then the same layer all-SQ and all-VQ-64.  TFLOP/s over the layer (2*M*oc*ic per matrix) and the
    fraction of the measured bf16 peak."""
    import torch
    from paper_2505_03803_b200 import binding as B
    peak, kind = measured_bf16_peak()
    out = {}
    hybrid = prefill_formats()
    for label, formats in (("hybrid", hybrid), ("all_sq", ["sq"] * 8), ("all_vq64", ["vq"] * 8)):
        mats = _prefill_layer(formats, M)
        ms, flops, tf = _time_prefill_layer(mats, M, reps)
        out[label] = (ms, flops, tf, sum(1 for m in mats if m[0].method == B.RWKVQ_SQ), len(mats))
        del mats
        torch.cuda.empty_cache()
    ms, flops, tf, n_sq, n = out["hybrid"]
    assert 0 < n_sq < n
    return {"workload": f"one 7B-class layer (8 projections, d=4096 h=14336), M={M} tokens, hybrid SQ/VQ-64, bf16 x bf16 -> fp32",
            "ms_per_layer": ms, "flop_per_layer": flops, "launches_per_layer": 2, "sq_matrices": n_sq,
            "formats": hybrid,
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                         "traffic": None, "peak_kind": f"of {kind} (burst)", "kernel": "prefill_kernel",
                         "frac_of_2250_nominal": tf / 2250.0},
            "all_sq": {"ms_per_layer": out["all_sq"][0], "tflops": out["all_sq"][2], "frac": out["all_sq"][2] / peak},
            "all_vq64": {"ms_per_layer": out["all_vq64"][0], "tflops": out["all_vq64"][2], "frac": out["all_vq64"][2] / peak}}


def proxy_leg(reps: int = 10, with_oracle: bool = True):
    """The proxy pass (Section 4.1) on fp16 matrices resident on the device: rwkvq_proxy_select over one
    matrix at a time (histogram of the 65 536 bit patterns = the sort of Eq. 5 as a counting sort, then the
    walk over the occupied bins, then the copy of the two numbers to the host), timed with events around
    the call.  A 256 x 256 matrix gives the fixed cost of the call (clear, walk, copy, synchronization);
    the large matrices minus that are the streaming pass, whose algorithmic traffic is 2 bytes per
    weight.  The oracle's sort-and-difference on the same values is timed beside it."""
    import torch
    from paper_2505_03803_b200 import binding as B
    from paper_2505_03803_b200 import stack as stack_mod
    peak, kind = measured_hbm_peak()
    ws = torch.empty(B.rwkvq_proxy_workspace_bytes(1), dtype=torch.uint8, device="cuda")

    def timed(w):
        B.rwkvq_proxy_select([w], 4, math.inf, math.inf, ws)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            pc, pf, _ = B.rwkvq_proxy_select([w], 4, math.inf, math.inf, ws)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps, float(pc[0]), float(pf[0])
    small = stack_mod.gen_weight_device(11, 256, 256, "gauss")
    fixed_ms, _, _ = timed(small)
    rows = []
    for (oc, ic, kind_w) in ((4096, 4096, "gauss"), (14336, 4096, "gauss"), (4096, 4096, "student")):
        w = stack_mod.gen_weight_device(12 + oc, oc, ic, kind_w)
        ms, pc, pf = timed(w)
        stream_ms = max(1e-6, ms - fixed_ms)
        gbs = 2.0 * oc * ic / (stream_ms * 1e-3) / 1e9
        rows.append({"matrix": f"{oc}x{ic} {kind_w}", "call_ms": ms, "histogram_ms": stream_ms, "P_c": pc, "P_f": pf,
                     "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                  "traffic": None, "peak_kind": f"of {kind}", "kernel": "proxy_hist_kernel",
                                  "algorithmic_bytes_per_launch": 2 * oc * ic}})
        if with_oracle and oc == 4096 and kind_w == "gauss":
            from oracle import rwkvq_oracle as orc
            wh = w.cpu().numpy().astype(np.float64)
            t0 = time.perf_counter()
            orc.proxy(wh, 4)
            rows[-1]["oracle_s"] = time.perf_counter() - t0
        del w
    return {"workload": "rwkvq_proxy_select on one fp16 matrix resident on the device, K = 4", "fixed_call_ms": fixed_ms,
            "fixed_call": "256 x 256 matrix: workspace clear, proxy_reduce_kernel, copy of the results, synchronization",
            "matrices": rows}


def vq_alu_roofline(oc, ic, entries, iters, ms, sm_mhz=1965.0, sms=148):
    """vq_kmeans_kernel against the fp32 instruction rate: an assignment pass evaluates, per (2-D vector,
    centre) pair, two subtractions, a multiply, a fused multiply-add and a compare-and-keep = 5 thread
    instructions; k-means++ seeding makes `entries` such passes against one new centre each (5 instructions per
    vector and pass) and every Lloyd iteration one pass against all centres.  Peak = 128 fp32 lanes per SM per
    clock at the maximum SM clock.  Centre updates, the scans of the seeding and the final fp64 assignment are
    not counted, so the fraction is a lower bound on how busy the lanes are."""
    vectors = oc * ic // 2
    work = 5.0 * vectors * entries * (iters + 1)          # iterations against all centres + the seeding passes
    achieved = work / (ms * 1e-3) / 1e12
    peak = sms * 128 * sm_mhz * 1e6 / 1e12
    return {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "T thread-instructions/s", "frac": achieved / peak,
            "traffic": None, "kernel": "vq_kmeans_kernel"}


def quantize_leg(reps: int = 5):
    """The device quantizers on one 7B-class layer: every projection scalar-quantized (Eq. 2) from fp16
    weights resident on the device, timed over the layer, and one 4096 x 4096 matrix vector-quantized
    (Eq. 3, 256 tiles, 64 entries, 10 Lloyd iterations).  The scalar quantizer reads 2 bytes and writes
    0.40625 bytes per weight: an HBM-bound kernel."""
    import torch
    from paper_2505_03803_b200 import binding as B
    from paper_2505_03803_b200 import inputs
    sp = inputs.STACKS["c3_7b"]
    gen = torch.Generator(device="cuda").manual_seed(1234)
    ws = torch.zeros(B.rwkvq_quantize_workspace_bytes(), dtype=torch.uint8, device="cuda")
    mats = []
    for (name, oc, ic, has_mu, stage) in inputs.layer_shapes(sp["d"], sp["h"]):
        w = (torch.randn((oc, ic), generator=gen, device="cuda") * 0.02).to(torch.float16)
        d = B.rwkvq_desc_for(oc, ic, B.RWKVQ_SQ, 3)
        mats.append((w, oc, ic, torch.empty(int(d.image_bytes), dtype=torch.uint8, device="cuda")))

    def layer():      # eight kernels enqueued back to back, one check (and synchronization) per layer
        for (w, oc, ic, img) in mats:
            B.rwkvq_quantize_dev_async(w, oc, ic, B.RWKVQ_SQ, 3, img, ws)
        if B.rwkvq_quantize_check(ws) != 0:
            raise SystemExit("bench.py: the quantizer leg saw a non-finite weight")
    layer()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        layer()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    weights = sum(oc * ic for (_w, oc, ic, _i) in mats)
    nbytes = sum(2 * oc * ic + img.numel() for (_w, oc, ic, img) in mats)
    gbs = nbytes / (ms * 1e-3) / 1e9
    peak, kind = measured_hbm_peak()
    w, oc, ic, _ = mats[0]
    dv = B.rwkvq_desc_for(oc, ic, B.RWKVQ_VQ, 6)
    imgv = torch.empty(int(dv.image_bytes), dtype=torch.uint8, device="cuda")
    B.rwkvq_quantize_dev(w, oc, ic, B.RWKVQ_VQ, 6, imgv, ws)
    torch.cuda.synchronize()
    e0.record()
    B.rwkvq_quantize_dev(w, oc, ic, B.RWKVQ_VQ, 6, imgv, ws)
    e1.record()
    torch.cuda.synchronize()
    vq_ms = e0.elapsed_time(e1)
    return {"workload": "one 7B-class layer (8 projections, d=4096 h=14336), fp16 weights on the device -> packed images",
            "sq_ms_per_layer": ms, "sq_weights_per_s": weights / (ms * 1e-3), "launches_per_layer": 2 * len(mats),
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak, "traffic": None,
                         "peak_kind": f"of {kind}", "kernel": "sq_quantize_kernel", "algorithmic_bytes_per_layer": nbytes,
                         "timed": "eight rwkvq_quantize_dev_async calls and one rwkvq_quantize_check (a stream "
                                  "synchronization) per layer"},
            "vq": {"matrix": f"{oc}x{ic}, 64 entries, 10 Lloyd iterations", "ms": vq_ms, "tiles": (oc // 256) * (ic // 256),
                   "weights_per_s": oc * ic / (vq_ms * 1e-3), "roofline": vq_alu_roofline(oc, ic, 64, 10, vq_ms)}}


def block_leg(configs=(("c3_7b", 1), ("c4_14b", 16)), max_steps=300, steps=None):
    """Whole blocks with their element-wise operators inside the same persistent launch (Appendix A.1 Eqs.
    20-27: token shift, R/K/V, WKV recurrence and sigmoid gate, O, channel-mix K/R, squared ReLU, V, output
    gate; plus the root-mean-square normalisation the chain needs), so that every stage reads what the stage
    before wrote: tokens/s of the chain of blocks, one token per sequence per step.  The matrix set is the
    appendix's (no gate matrix), the shapes and depth those of the named stack."""
    import torch
    from paper_2505_03803_b200 import binding as B
    from paper_2505_03803_b200 import inputs, stack as stack_mod
    peak, kind = measured_hbm_peak()
    out = {}
    for (wl, batch) in configs:
        sp = inputs.STACKS[wl]
        st = stack_mod.BlockStack(sp["d"], sp["h"], sp["layers"], sp["entries"], batch, n_outliers=sp["outliers"], tag=wl)
        st.set_token(11)
        for _ in range(3):
            st.run_step_host()
        torch.cuda.synchronize()
        K = steps if steps is not None else int(min(max_steps, max(20, 1500.0 / max(0.05, st.stream_bytes / 2.0e9))))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(K):
            st.run_step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / K
        stream = torch.cuda.current_stream()
        e0.record()
        for _ in range(K):
            st.run_step_host(stream)
            stream.synchronize()
        e1.record()
        torch.cuda.synchronize()
        ms_e2e = e0.elapsed_time(e1) / K
        if B.rwkvq_device_status() != 0:
            raise SystemExit("bench.py: a device-side wait timed out in the block leg")
        finite = bool(torch.isfinite(st.out_v).all())
        alg = st.stream_bytes + st.act_bytes
        gbs = alg / (ms * 1e-3) / 1e9
        out[f"{wl}_b{batch}"] = {
            "tokens_per_s": batch / (ms * 1e-3), "ms_per_step": ms, "steps": K, "matrices": len(st.ops), "sq_matrices": st.n_sq,
            "stages": st.n_stages, "packed_bytes_per_step": st.stream_bytes, "activation_bytes_per_step": st.act_bytes,
            "outputs_finite": finite, "setup_s": round(st.setup_s, 1),
            "e2e": {"value": batch / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(st.x0_host.numel() * 2),
                    "d2h_bytes_per_step": int(st.out_host.numel() * 4)},
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak, "traffic": None,
                         "peak_kind": f"of {kind}", "kernel": "step_kernel", "algorithmic_bytes_per_launch": alg}}
        del st
        torch.cuda.empty_cache()
    return {"workload": "chain of RWKV blocks (7 projections per block, element-wise operators fused into the step), "
                        "one token per sequence per step", "configs": out}


# ---------------------------------------------------------------------------------------------
# GPU leg
# ---------------------------------------------------------------------------------------------
def build_stack(args, workload, batch, force_method=None, distinct_layers=None):
    from paper_2505_03803_b200 import binding as B
    from paper_2505_03803_b200 import inputs, stack as stack_mod
    sp = inputs.STACKS[workload]
    fm = force_method or args.force_method
    force = None if fm is None else (B.RWKVQ_SQ if fm == "sq" else B.RWKVQ_VQ)
    weights = args.weights or ("device" if args.quantizer == "device" else "host")
    t0 = time.time()
    st = stack_mod.Stack(sp["d"], sp["h"], sp["layers"], sp["entries"], batch, n_outliers=sp["outliers"],
                         tag=workload, device="cuda", distinct_layers=args.distinct_layers if distinct_layers is None else distinct_layers,
                         force_method=force,
                         quantizer=args.quantizer, weights=weights)
    st.bench_setup_s = time.time() - t0
    return st


def measure_stack(st, args, workload, K, W, world, dist, gpu_id, with_e2e=True):
    """W warm-up steps, then K timed steps of one stack at its current batch: device-resident timing
    with one event per step boundary, then the end-to-end loop through rwkvq_step_run_host; clocks are
    sampled over both."""
    import torch
    from paper_2505_03803_b200 import binding as B
    batch = st.batch
    if args.stage_group > 0:
        for i, o in enumerate(st.ops):
            o.stage = i // args.stage_group
        st.n_stages = len({o.stage for o in st.ops})
    if args.mode == "step":
        st.plan_step()
    run = st.run_step if args.mode == "step" else st.run_ops
    launches_per_step = 1 if args.mode == "step" else len(st.ops)
    stream = torch.cuda.current_stream()
    for _ in range(W):
        run(stream)
    torch.cuda.synchronize()
    if B.rwkvq_device_status() != 0:
        raise SystemExit("bench.py: a device-side wait timed out during warm-up")
    sampler = ClockSampler(gpu_id)
    sampler.start()
    time.sleep(0.3)

    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    ev[0].record(stream)
    for i in range(K):
        run(stream)
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    total_ms = ev[0].elapsed_time(ev[K])
    per_launch_ms = [ev[i].elapsed_time(ev[i + 1]) / launches_per_step for i in range(K)]
    status = B.rwkvq_device_status()

    # ---- end to end: activations from pinned host memory, results back to the host, every step
    def e2e_region():
        for _ in range(3):
            st.run_step_host(stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(K):
            st.run_step_host(stream)
            stream.synchronize()          # the caller reads the step's outputs before the next step
        b.record(stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return a.elapsed_time(b)

    e2e_ms, e2e_copies = None, None
    if with_e2e and args.mode == "step":
        e2e_ms = e2e_region()
        e2e_copies = "plain order" if os.environ.get("RWKVQ_HOST_OVERLAP", "")[:1] == "0" else \
            "overlapped with the step where the step copies 8 MB or more"
        if world == 1 and status == 0 and e2e_copies != "plain order" and B.rwkvq_device_status() != 0:
            # the overlapped host-buffer step gave up on a bounded wait: measure the plain order instead
            print("bench.py: the overlapped host-buffer step timed out; end-to-end figure taken in the plain order",
                  file=sys.stderr)
            os.environ["RWKVQ_HOST_OVERLAP"] = "0"
            e2e_ms = e2e_region()
            e2e_copies = "plain order (the overlapped order timed out on this machine)"
    t2 = time.time()
    clocks = sampler.stop(t0, t2)
    if status != 0 or B.rwkvq_device_status() != 0:
        raise SystemExit("bench.py: a device-side wait timed out during the timed region")

    max_ms, tokens = aggregate_over_ranks(total_ms, float(batch * K), dist if world > 1 else None)
    e2e = None
    if e2e_ms is not None:
        m2, tok2 = aggregate_over_ranks(e2e_ms, float(batch * K), dist if world > 1 else None)
        e2e = {"value": tok2 / (m2 * 1e-3), "unit": UNIT, "copies": e2e_copies, "h2d_bytes_per_step": int(st.act_host.numel()),
               "d2h_bytes_per_step": int(st.y_host.numel())}
    peak, peak_kind = measured_hbm_peak()
    alg_bytes = st.stream_bytes + st.act_bytes
    avg_launch_ms = sum(per_launch_ms) / len(per_launch_ms)
    achieved = alg_bytes / launches_per_step / (avg_launch_ms * 1e-3) / 1e9
    traffic = None
    if (NCU_TRAFFIC_PER_ALGORITHMIC_BYTE is not None and args.mode == "step" and args.stage_group == 0
            and args.force_method is None):
        traffic = int(NCU_TRAFFIC_PER_ALGORITHMIC_BYTE * alg_bytes)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_kind": f"of {peak_kind}",
                "kernel": "step_kernel" if args.mode == "step" else "gemv_kernel",
                "algorithmic_bytes_per_launch": alg_bytes / launches_per_step,
                "launch_ms_avg": avg_launch_ms, "launch_ms_median": statistics.median(per_launch_ms),
                "launch_ms_min": min(per_launch_ms), "frac_of_8TBs_nominal": achieved / 8000.0}
    config = {"workload": workload_name(workload, batch), "batch": batch, "mode": args.mode,
              "matrices": len(st.ops), "sq_matrices": st.n_sq, "stages": st.n_stages,
              "weights": st.n_weights, "packed_bytes_per_step": st.stream_bytes,
              "activation_bytes_per_step": st.act_bytes, "distinct_layers": st.n_src, "quantizer": st.quantizer,
              "weights_drawn_on": st.weights, "stage_group": args.stage_group,
              "l2": "inputs larger than L2: every step streams the whole packed stack once",
              "not_included": "WKV recurrence, norms, gates, embedding and head are not part of the workload",
              "tau_c": st.tau_c, "setup_s": round(st.bench_setup_s, 1)}
    return {"value": tokens / (max_ms * 1e-3), "ms_per_step": max_ms / K, "steps": K, "warmup": W, "roofline": roofline,
            "e2e": e2e, "clocks": clocks, "gpu_launches": K * launches_per_step, "config": config}


def default_steps(st, args):
    est_ms = max(0.05, st.stream_bytes / 2.0e9)    # ms per step at 2 TB/s: only sizes the default step count
    K = args.steps if args.steps is not None else int(min(2000, max(20, 2000.0 / est_ms)))
    W = max(args.warmup if args.warmup is not None else 5, 3)
    return K, W


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2505_03803_b200 import binding as B
    from paper_2505_03803_b200 import build as build_mod
    from paper_2505_03803_b200 import inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; this benchmark has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build_mod.build()
    if world > 1:
        dist.barrier()
    B.lib()
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        gpu_id = str(local_rank)

    whole = args.workload is None
    workload = args.workload or HEADLINE[0]
    batch = args.batch or (HEADLINE[1] if whole else inputs.STACKS[workload]["batches"][0])
    st = build_stack(args, workload, batch)
    K, W = default_steps(st, args)
    head = measure_stack(st, args, workload, K, W, world, dist, gpu_id)
    head["config"]["replicas"] = "independent replica per GPU, no exchange step" if world > 1 else "single GPU"
    del st
    torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    configs = None
    if whole and world == 1 and not args.no_configs:
        configs, st, cur = {}, None, None
        for (wl, b) in CONFIGS:
            if cur != wl:
                del st
                torch.cuda.empty_cache()
                st, cur = build_stack(args, wl, b), wl
            else:
                st.set_batch(b)
            k, w = default_steps(st, args)
            r = measure_stack(st, args, wl, k, w, 1, None, gpu_id)
            configs[f"{wl}_b{b}"] = {"tokens_per_s": r["value"], "ms_per_step": r["ms_per_step"], "steps": r["steps"],
                                     "roofline": r["roofline"], "clocks": r["clocks"], "e2e": r["e2e"],
                                     "config": r["config"]}
        del st
        torch.cuda.empty_cache()

    # each format alone on the headline stack, so that neither hides behind the mix (two distinct layers,
    # reused: the set-up of 488 k-means matrices is not what is timed; 180 MB of images still exceed L2)
    formats = None
    if whole and world == 1 and not args.no_configs and args.force_method is None:
        formats = {}
        for fm in ("sq", "vq"):
            st = build_stack(args, workload, batch, force_method=fm, distinct_layers=2)
            k, w = default_steps(st, args)
            r = measure_stack(st, args, workload, min(k, 200), w, 1, None, gpu_id, with_e2e=False)
            formats["all_" + fm] = {"tokens_per_s": r["value"], "ms_per_step": r["ms_per_step"], "steps": r["steps"],
                                    "roofline": r["roofline"], "clocks": r["clocks"],
                                    "packed_bytes_per_step": r["config"]["packed_bytes_per_step"],
                                    "distinct_layers": 2}
            del st
            torch.cuda.empty_cache()

    prefill = prefill_leg() if world == 1 and not args.no_prefill else None
    quantize = quantize_leg() if world == 1 and not args.no_quantize else None
    proxy = proxy_leg(with_oracle=not args.no_cpu_baseline) if world == 1 and not args.no_proxy else None
    block = block_leg(steps=args.steps) if world == 1 and whole and not args.no_block else None

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        sp = inputs.STACKS[workload]
        r = time_oracle(workload, batch, budget_s=12.0)
        cpu = {"value": r["value"], "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
               "sample": (f"the oracle's decode + token shift + fp64 product over the 8 matrices of one layer "
                          f"({r['sample_weights']} of {r['total_weights']} weights), {r['n']} repetitions, "
                          f"{r['per_sample_s']:.3f} s each, scaled to {sp['layers']} layers")}

    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": head["steps"],
        "warmup": head["warmup"], "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16", "data": "synthetic", "config": head["config"],
        "roofline": head["roofline"], "cpu_baseline": cpu, "e2e": head["e2e"], "clocks": head["clocks"],
        "gpu_launches": head["gpu_launches"], "hbm_gbs": head["roofline"]["achieved"],
        "configs": configs, "formats": formats, "prefill": prefill, "quantize": quantize, "proxy": proxy, "block": block,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def main(argv=None):
    args = parse_args(argv)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
