#!/usr/bin/env python
"""Benchmark of the MoE feed-forward layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--all] [--impl reference]

One step = one forward pass of the whole layer (router, top-k gating, grouping, expert FFN,
gate-weighted combine) over one batch of seeded synthetic input.  The default workload is the
phone-scale layer at batch-1 decode (the largest single-GPU decode configuration); steps walk a ring of
distinct layers whose touched weights exceed the L2 several times over, so every step reads its experts
from HBM.  Prints ONE JSON line; unless --no-others is given it also times the other configurations
(decode and prefill, dense and weight-decomposed experts, a shortened offload stack) and reports them
under "others", each with its roofline.  N > 1: independent replicas, one per GPU, no collective.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from synth import workloads as W  # noqa: E402

L2_BYTES = 126 * 1024 * 1024

WORKLOADS = {
    # name: (shape, T, kind)
    "wearable-decode-T1": (W.WEARABLE, 1, "decode"),
    "wearable-decode-T8": (W.WEARABLE, 8, "decode"),
    "wearable-prefill-T512": (W.WEARABLE, 512, "prefill"),
    "phone-decode-T1": (W.PHONE, 1, "decode"),
    "phone-prefill-T2048": (W.PHONE, 2048, "prefill"),
    "phone-wd128-decode-T1": (W.PHONE_WD128, 1, "decode"),
    "phone-wd1024-decode-T1": (W.PHONE_WD1024, 1, "decode"),
    "phone-wd128-prefill-T2048": (W.PHONE_WD128, 2048, "prefill"),
    "phone-wd1024-prefill-T2048": (W.PHONE_WD1024, 2048, "prefill"),
    "tiny-T16": (W.TINY, 16, "decode"),
}
DEFAULT = "phone-decode-T1"
# timed after the main workload and reported under "others" (the offload stack, shortened, is added to them)
OTHERS = ["wearable-decode-T1", "wearable-decode-T8", "wearable-prefill-T512", "phone-prefill-T2048",
          "phone-wd128-decode-T1", "phone-wd1024-decode-T1", "phone-wd128-prefill-T2048", "phone-wd1024-prefill-T2048"]
NOMINAL = {"hbm_gbs": 8000.0, "tflops": 2250.0}   # the target's denominators: about 8 TB/s, dense bf16 2.25 PFLOP/s

# Shape sweep (--sweep): batch-1 decode over the paper's ablation grid -- active experts k in {1, 2, 4, 8} at E = 8,
# total experts E in {2, 4, 8, 16} at k = 2 (Fig. 7: time grows with k, not with E) -- and the paper's own layer
# widths (Table 1).  Reported under "sweep"; not part of --all.
SWEEP = {}
for _k in (1, 2, 4, 8):
    SWEEP[f"sweep-k{_k}-E8"] = (W.WEARABLE.with_(name=f"wearable k={_k} E=8", top_k=_k), 1, "decode")
for _E in (2, 4, 16):
    SWEEP[f"sweep-k2-E{_E}"] = (W.WEARABLE.with_(name=f"wearable k=2 E={_E}", n_experts=_E), 1, "decode")
SWEEP["sweep-d1440-f3840"] = (W.LayerShape("paper phone widths", 8, 1440, 3840), 1, "decode")
SWEEP["sweep-d432-f1280"] = (W.LayerShape("paper wearable widths", 8, 432, 1280), 1, "decode")
WORKLOADS.update(SWEEP)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        m = json.load(open(p))
        return {"hbm_gbs": m["hbm_gbs"], "tflops": m["bf16_tflops"], "tflops_sustained": m["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def algorithmic_bytes(shape: W.LayerShape, n_active_experts: float, T: int) -> float:
    """Bytes one layer forward must move: the selected experts' weights once, the router, x and y."""
    d, E = shape.d_model, shape.n_experts
    return n_active_experts * W.expert_bytes(shape) + 2 * d * E + 2 * 2 * T * d


def flops(shape: W.LayerShape, T: int) -> float:
    per = 6 * shape.wd_rank * (shape.d_model + shape.d_ff) if shape.wd_rank else 6 * shape.d_model * shape.d_ff
    return float(T) * shape.top_k * per + 2.0 * T * shape.d_model * shape.n_experts


def build_ring(shape, T, device, min_touched_bytes, ring_override=0):
    """Distinct layers (weights + inputs) so that consecutive steps never find their experts in L2."""
    import paper_2503_00245_b200 as P
    touched = min(shape.n_experts, T * shape.top_k) * W.expert_bytes(shape)
    n_layers = max(2, -(-min_touched_bytes // touched))
    n_layers = min(n_layers, 64)
    if ring_override:
        n_layers = ring_override
    kw = dict(d_model=shape.d_model, d_ff=shape.d_ff, n_experts=shape.n_experts, top_k=shape.top_k)
    ring = []
    for l in range(n_layers):
        t = W.make_layer(shape, T, device=device, layer=l)
        lay = P.MoELayer.from_math_layout(kw, t, x_dtype=t["x"].dtype, max_tokens=T)
        x = t["x"]
        ring.append({"layer": lay, "x": x, "y": torch.empty_like(x),
                     "idx": torch.empty((T, shape.top_k), dtype=torch.int32, device=device),
                     "w": torch.empty((T, shape.top_k), dtype=torch.float32, device=device)})
        del t
    torch.cuda.synchronize()
    return ring


def run_ring(ring, steps, start=0):
    n = len(ring)
    for i in range(steps):
        r = ring[(start + i) % n]
        r["layer"].forward(r["x"], y=r["y"], topk_idx=r["idx"], topk_w=r["w"])


def time_workload(name, steps, warmup, device, rank, world, ring_override=0, use_graph=True, min_ms=1500.0):
    shape, T, kind = WORKLOADS[name]
    pk = peaks()
    ring = build_ring(shape, T, device, 4 * L2_BYTES, ring_override)
    n = len(ring)
    stream = torch.cuda.current_stream()
    launches0 = sum(_launches(r) for r in ring)
    run_ring(ring, max(warmup, 3))
    torch.cuda.synchronize()
    for r in ring:
        assert r["layer"].check() == 0, "a kernel flagged an error during warm-up"
    launches_per_step = (sum(_launches(r) for r in ring) - launches0) / max(warmup, 3)

    # CUDA graph of one trip around the ring (decode steps are launch-bound otherwise)
    graph = None
    mode = "stream"
    if use_graph:
        try:
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                run_ring(ring, n)
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=side):
                    run_ring(ring, n)
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            graph, mode = g, "cuda_graph"
        except Exception as e:  # noqa: BLE001
            sys.stderr.write(f"[bench] CUDA graph capture unavailable ({e}); timing plain launches\n")
            torch.cuda.synchronize()
            graph = None
    # whole trips around the ring, rounded up; the same trips are repeated until the timed region is long enough
    # for the clock samplers (this one and any outside) to see the load
    trips = -(-steps // n)
    steps_trip = trips * n

    def timed_region(n_trips):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()
        e0.record()
        if graph is not None:
            for _ in range(n_trips):
                graph.replay()
        else:
            run_ring(ring, n_trips * n)
        e1.record()
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        return e0.elapsed_time(e1)

    # one untimed region of the steps asked for tells how many repeats make the timed region long enough; the
    # timed region is then ONE bracket (barrier + synchronise on both sides) around all of them
    reps = 1
    if world == 1 and min_ms > 0:   # replicas keep to the steps asked for: every rank runs the same region
        reps = max(1, int(-(-min_ms // max(timed_region(trips), 1e-3))))
    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    if sampler:
        sampler.start()
    ms = timed_region(trips * reps)
    clocks = sampler.stop() if sampler else None
    steps_eff = steps_trip * reps
    for r in ring:
        assert r["layer"].check() == 0, "a kernel flagged an error during the timed region"

    # distinct experts actually read per step (exact, from the routing the kernels produced)
    act = sum(len(set(r["idx"].flatten().tolist())) for r in ring) / n
    res = {"name": name, "shape": shape, "T": T, "kind": kind, "ms_total": ms, "steps": steps_eff,
           "ms_per_step": ms / steps_eff, "launch_mode": mode, "ring_layers": n, "active_experts_per_step": act,
           "launches_per_step": launches_per_step, "clocks": clocks, "peaks": pk, "ring": ring}
    return res


def _launches(r):
    from paper_2503_00245_b200 import binding as B
    return B.moe_launch_count(r["layer"].ctx)


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel come from the ncu summaries under
# profiles/ (same workload, ring of fewer layers).  A summary carries the lines
#     traffic_bytes_per_launch: <bytes>
#     kernel_source: <file under csrc/> sha256 <hex>
# and its figure is used only while that source file is unchanged: once the kernel has been edited the counters
# no longer describe it and "traffic" is null until the capture is retaken.
PROFILE_OF = {
    "wearable-decode-T1": "dense_stream_kernel_wearable_decode_T1.md",
    "wearable-decode-T8": "dense_stream_kernel_wearable_decode_T8.md",
    "phone-decode-T1": "dense_stream_kernel_phone_decode_T1.md",
    "phone-prefill-T2048": "grouped_gemm_kernel_phone_prefill_T2048.md",
    "phone-wd128-decode-T1": "wd_decode_kernel_phone_wd128_decode_T1.md",
    "phone-wd1024-decode-T1": "wd_stream_kernel_phone_wd1024_decode_T1.md",
}


def ncu_traffic(name):
    import hashlib
    import re
    fn = PROFILE_OF.get(name)
    path = os.path.join(ROOT, "profiles", fn) if fn else None
    if not path or not os.path.exists(path):
        return None
    text = open(path).read()
    m = re.search(r"^traffic_bytes_per_launch:\s*(\d+)", text, re.M)
    k = re.search(r"^kernel_source:\s*(\S+)\s+sha256\s+([0-9a-f]{64})", text, re.M)
    if not m or not k:
        return None
    src = os.path.join(ROOT, "paper_2503_00245_b200", "csrc", k.group(1))
    if not os.path.exists(src) or hashlib.sha256(open(src, "rb").read()).hexdigest() != k.group(2):
        return None
    return int(m.group(1))


def roofline(res):
    r = _roofline(res)
    r["traffic"] = ncu_traffic(res.get("name"))
    nominal = NOMINAL["hbm_gbs"] if r["bound"] == "hbm" else NOMINAL["tflops"]
    r["peak_nominal"] = nominal
    r["frac_nominal"] = round(r["achieved"] / nominal, 4)
    return r


def _decode_kernel_name(shape, T):
    """The kernel that streams the experts at this shape (the library's dispatch rule, restated for the label)."""
    if not shape.wd_rank:
        return "dense_stream_kernel"
    wd_bytes = shape.top_k * W.expert_bytes(shape)
    return ("wd_decode_kernel" if wd_bytes <= 32 * 1024 * 1024 else "wd_stream_kernel") if T == 1 else "stream_ffn_kernel"


def _roofline(res):
    shape, T, pk = res["shape"], res["T"], res["peaks"]
    sec = res["ms_per_step"] * 1e-3
    if res["kind"] == "decode":
        b = algorithmic_bytes(shape, res["active_experts_per_step"], T)
        ach = b / sec / 1e9
        return {"bound": "hbm", "achieved": round(ach, 1), "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": round(ach / pk["hbm_gbs"], 4), "traffic": None, "peak_source": pk["source"],
                "bytes_per_launch": int(b), "kernel": _decode_kernel_name(shape, T),
                "note": "duration = whole step (router + expert kernel) / 1"}
    fl = flops(shape, T)
    t_tc = fl / (pk["tflops_sustained"] * 1e12)
    t_hbm = algorithmic_bytes(shape, shape.n_experts, T) / (pk["hbm_gbs"] * 1e9)
    if t_hbm > t_tc:
        b = algorithmic_bytes(shape, shape.n_experts, T)
        ach = b / sec / 1e9
        return {"bound": "hbm", "achieved": round(ach, 1), "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": round(ach / pk["hbm_gbs"], 4), "traffic": None, "peak_source": pk["source"],
                "tensor_tflops": round(fl / sec / 1e12, 1)}
    ach = fl / sec / 1e12
    return {"bound": "tensor", "achieved": round(ach, 1), "peak": pk["tflops_sustained"], "unit": "TFLOP/s",
            "frac": round(ach / pk["tflops_sustained"], 4), "traffic": None, "peak_source": pk["source"],
            "peak_kind": "sustained bf16 (kernel timed inside a long step)"}


def e2e_measure(res, steps):
    """Same metric through the public call with HOST buffers: pinned x -> device, layer, y -> host, per step."""
    ring = res["ring"]
    T, shape = res["T"], res["shape"]
    n = len(ring)
    hx = [r["x"].cpu().pin_memory() for r in ring]
    hy = [torch.empty_like(h).pin_memory() for h in hx]
    steps = min(steps, 2000)
    for i in range(min(8, steps)):
        r = ring[i % n]
        r["x"].copy_(hx[i % n], non_blocking=True)
        r["layer"].forward(r["x"], y=r["y"])
        hy[i % n].copy_(r["y"], non_blocking=True)
        torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(steps):
        r = ring[i % n]
        r["x"].copy_(hx[i % n], non_blocking=True)
        r["layer"].forward(r["x"], y=r["y"])
        hy[i % n].copy_(r["y"], non_blocking=True)
        torch.cuda.current_stream().synchronize()      # the caller reads y before the next token
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    nbytes = hx[0].numel() * hx[0].element_size()
    # decode on the streaming path: the finalising CTAs can store y straight into mapped pinned host memory, which
    # saves the device -> host copy (x still comes by a copy: every CTA reads it, from L2)
    mapped_ms = None
    if T <= 16 and not shape.wd_rank:
        for i in range(8):
            r = ring[i % n]
            r["x"].copy_(hx[i % n], non_blocking=True)
            r["layer"].forward(r["x"], y=hy[i % n])
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            r = ring[i % n]
            r["x"].copy_(hx[i % n], non_blocking=True)
            r["layer"].forward(r["x"], y=hy[i % n])
            torch.cuda.current_stream().synchronize()
        e1.record()
        torch.cuda.synchronize()
        mapped_ms = e0.elapsed_time(e1) / steps
    res["e2e_mapped_ms"] = mapped_ms
    return ms, nbytes, nbytes


def metric_of(res, ms_per_step, world=1):
    T = res["T"]
    if res["kind"] == "decode":
        return "moe_layer_us_per_token_decode", ms_per_step * 1e3 / (T * world), "us/token", False
    return "moe_layer_prefill_tokens_per_s", T * world / (ms_per_step * 1e-3), "tokens/s", True


def cpu_baseline(name, budget_s=12.0):
    """The CPU checker as it stands, timed on this machine's host cores on the same workload."""
    import numpy as np
    from threadpoolctl import threadpool_info
    from oracle import moe_oracle as O
    shape, T, kind = WORKLOADS[name]
    t = W.make_layer(shape, T, device="cpu", layer=0)
    h = {k: W.to_host_bits(v) for k, v in t.items()}
    ex = {k: v for k, v in h.items() if k not in ("x", "w_router", "b_router")}
    O.layer_forward(h["x"], h["w_router"], h["b_router"], ex, shape.top_k)
    n, t0 = 0, time.perf_counter()
    while True:
        O.layer_forward(h["x"], h["w_router"], h["b_router"], ex, shape.top_k)
        n += 1
        el = time.perf_counter() - t0
        if el > budget_s or n >= 2000:
            break
    per = el / n
    threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    if kind == "decode":
        val, unit = per * 1e6 / T, "us/token"
    else:
        val, unit = T / per, "tokens/s"
    return {"value": round(val, 3), "unit": unit, "cores": int(threads), "kind": "oracle",
            "sample": f"{n} forward passes of layer 0 of the ring ({el:.1f} s of CPU time), numpy fp64"}


def run_offload_stack(a, device, emit=True, fp8=False):
    """Stacked decode with host-resident experts: n_layers phone-scale layers (E = 16, top-2), `slots` experts
    per layer resident in HBM, the rest in pinned host memory, Zipf(1.2)-skewed routing; one step = one token
    through all layers.  Reports us/token and the host-link traffic against the measured pinned H2D rate."""
    import paper_2503_00245_b200 as P
    from paper_2503_00245_b200 import binding as B
    sh = W.PHONE_OFFLOAD
    n_layers, slots, steps = a.layers, a.slots, a.decode_steps
    layers = []
    for l in range(n_layers):
        r_w, r_b = W.make_router(sh, device, l)
        ex = W.make_experts(sh, device, l)
        layers.append({"w_router": r_w, "b_router": r_b, "gud": P.pack_dense(ex["w_gate"], ex["w_up"], ex["w_down"])})
        del ex
        if l % 4 == 3:
            torch.cuda.synchronize()
    def gen():
        for lay in layers:
            yield lay
            lay["gud"] = None          # the device copy is no longer needed once it is in pinned memory
    stack = P.OffloadedStack(sh.d_model, sh.d_ff, sh.n_experts, sh.top_k, slots, gen(), fp8=fp8)
    torch.cuda.empty_cache()
    # pinned host->device bandwidth of this machine (the roofline of a miss)
    probe_dst = torch.empty(stack.slot_bytes, dtype=torch.uint8, device=device)
    src = stack.host[0].view(torch.uint8).reshape(-1)[:stack.slot_bytes]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    probe_dst.copy_(src, non_blocking=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(8):
        probe_dst.copy_(src, non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    h2d_gbs = 8 * stack.slot_bytes / (e0.elapsed_time(e1) * 1e-3) / 1e9
    hs = [W.make_x(sh.with_(x_dtype="f32"), 1, device=device, step=s)[0].contiguous() for s in range(steps + 3)]
    for s in range(3):
        stack.step(hs[steps + s].clone())
    torch.cuda.synchronize()
    st0 = stack.stats()
    ht0 = B.moe_offload_host_times(stack.off)
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    trace = []
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0.record()
    for s in range(steps):
        trace.append(stack.step(hs[s]))
    e1.record()
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    clocks = sampler.stop()
    assert stack.check() == 0
    ms = e0.elapsed_time(e1)
    st1 = stack.stats()
    fetches, nbytes, hits = (st1[k] - st0[k] for k in ("fetches", "bytes", "hits"))
    lookups = steps * n_layers * sh.top_k
    # Eq. 4-5 on the routing the layers produced, per layer (B = layers, T = steps)
    tr = torch.tensor(trace, dtype=torch.int32, device=device).permute(1, 0, 2).contiguous()
    hsum = torch.zeros(1, dtype=torch.int64, device=device)
    B.moe_expert_replacements(tr, n_layers, steps, sh.top_k, sh.n_experts, hsum)
    torch.cuda.synchronize()
    exrep = (int(hsum.item()) // 2) / (n_layers * sh.top_k * max(1, steps - 1))
    # expert balance per layer (Section 3.3): mean over the layers of the deviation from the uniform share, percent
    cnt = torch.zeros((n_layers, sh.n_experts), dtype=torch.int64, device=device)
    dlt = torch.zeros(n_layers + 1, dtype=torch.float64, device=device)
    bad = torch.zeros(1, dtype=torch.int64, device=device)
    B.moe_delta_uniform(tr, n_layers, steps, sh.top_k, sh.n_experts, cnt, dlt, bad)
    torch.cuda.synchronize()
    delta_uniform = float(dlt[n_layers].item())
    ht1 = B.moe_offload_host_times(stack.off)
    us_tok = ms * 1e3 / steps
    bytes_tok = nbytes / steps
    t_link = bytes_tok / (h2d_gbs * 1e9) * 1e6
    t_hbm = n_layers * sh.top_k * W.expert_bytes(sh) / (peaks()["hbm_gbs"] * 1e9) * 1e6
    line = {
        "metric": "moe_stack_us_per_token_decode_offload", "value": round(us_tok, 2), "unit": "us/token",
        "n_gpus": 1, "steps": steps, "warmup": 3, "ms_per_step": round(ms / steps, 4), "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 weights/activations, f32 accumulate",
        "data": "synthetic",
        "config": {"workload": "phone-offload-stack-fp8" if fp8 else "phone-offload-stack", "shape": W.describe(sh),
                   "host_copies": "FP8 E4M3 codes + fp32 row scales" if fp8 else "bf16", "layers": n_layers,
                   "resident_slots_per_layer": slots, "T": 1, "decode_steps": steps,
                   "launch_mode": "stream (the host polls a mapped routing word per layer)",
                   "l2": "inputs larger than L2: 24 distinct layers per token"},
        "roofline": {"bound": "host_link", "achieved": round(bytes_tok / (us_tok * 1e-6) / 1e9, 2),
                     "peak": round(h2d_gbs, 2), "unit": "GB/s",
                     "frac": round(t_link / us_tok, 4), "traffic": None,
                     "peak_source": "pinned H2D copy of one expert, measured in this run",
                     "note": "frac = (fetch bytes / measured H2D rate) / time per token"},
        "offload": {"fetch_bytes_per_token": int(bytes_tok), "fetches_per_token": round(fetches / steps, 3),
                    "hit_rate": round(hits / lookups, 4), "exrep": round(exrep, 4),
                    "delta_uniform_pct": round(delta_uniform, 3),
                    "no_miss_floor_us": round(t_hbm, 1), "host_link_floor_us": round(t_link, 1),
                    "host_wall_us_per_token": round(wall * 1e6 / steps, 1),
                    # where a token's time goes besides the link: the host waiting for routing words (the device is
                    # then computing the layer's last chunk and the next layer's norm + router) and queueing work
                    "host_poll_us_per_token": round((ht1["poll_s"] - ht0["poll_s"]) * 1e6 / steps, 1),
                    "host_issue_us_per_token": round((ht1["issue_s"] - ht0["issue_s"]) * 1e6 / steps, 1),
                    "link_idle_us_per_token": round(us_tok - t_link, 1)},
        "e2e": {"value": round(wall * 1e6 / steps, 2), "unit": "us/token", "h2d_bytes_per_step": int(bytes_tok),
                "d2h_bytes_per_step": n_layers * sh.top_k * 4},
        "gpu_launches": int(B.moe_launch_count(stack.ctx)),
        "clocks": clocks,
    }
    stack.close()
    del stack
    torch.cuda.empty_cache()
    if emit:
        print(json.dumps(line))
        return 0
    return line


def run_offload_eq8(a, device):
    """The paper's offload rule itself (Eq. 8: as many device slots as active experts, E = 8, top-2) on phone-scale
    layers, driven by synthetic sticky routing traces whose expert replacement ratio (Eq. 4-5) is set to the two
    levels the paper reports for its models without and with the block-wise selection loss (Table 3).  The expert
    sets are known to the host, so a layer's misses are copied while earlier layers compute."""
    import paper_2503_00245_b200 as P
    from paper_2503_00245_b200 import binding as B
    sh = W.PHONE.with_(name="phone-eq8", bias="none")
    n_layers, steps = a.layers, min(a.decode_steps, 64)
    layers = []
    for l in range(n_layers):
        r_w, r_b = W.make_router(sh, device, l)
        ex = W.make_experts(sh, device, l)
        layers.append({"w_router": r_w, "b_router": r_b, "gud": P.pack_dense(ex["w_gate"], ex["w_up"], ex["w_down"])})
        del ex
        if l % 4 == 3:
            torch.cuda.synchronize()

    def gen():
        for lay in layers:
            yield lay
            lay["gud"] = None

    stack = P.OffloadedStack(sh.d_model, sh.d_ff, sh.n_experts, sh.top_k, sh.top_k, gen())
    torch.cuda.empty_cache()
    probe_dst = torch.empty(stack.slot_bytes, dtype=torch.uint8, device=device)
    src = stack.host[0].view(torch.uint8).reshape(-1)[:stack.slot_bytes]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    probe_dst.copy_(src, non_blocking=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(8):
        probe_dst.copy_(src, non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    h2d_gbs = 8 * stack.slot_bytes / (e0.elapsed_time(e1) * 1e-3) / 1e9
    hs = [W.make_x(sh.with_(x_dtype="f32"), 1, device=device, step=s)[0].contiguous() for s in range(steps)]
    runs = []
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    for label, target in (("without block-wise selection", 0.4382), ("with block-wise selection", 0.0655)):
        p_stay = 1.0 - target * sh.top_k          # one member replaced per change: ExRep = (1 - p_stay) / k
        traces = [W.sticky_routing_trace(4242 + l, steps + 1, sh.n_experts, sh.top_k, p_stay).tolist()
                  for l in range(n_layers)]
        stack.step_trace(hs[0].clone(), [traces[l][0] for l in range(n_layers)])   # warm-up: brings in the first sets
        torch.cuda.synchronize()
        st0 = stack.stats()
        t0 = time.perf_counter()
        e0.record()
        for s_ in range(steps):
            stack.step_trace(hs[s_], [traces[l][s_ + 1] for l in range(n_layers)])
        e1.record()
        torch.cuda.synchronize()
        wall = time.perf_counter() - t0
        assert stack.check() == 0
        ms = e0.elapsed_time(e1)
        st1 = stack.stats()
        nbytes = st1["bytes"] - st0["bytes"]
        tr = torch.tensor([t[1:] for t in traces], dtype=torch.int32, device=device).contiguous()
        hsum = torch.zeros(1, dtype=torch.int64, device=device)
        B.moe_expert_replacements(tr, n_layers, steps, sh.top_k, sh.n_experts, hsum)
        torch.cuda.synchronize()
        exrep = (int(hsum.item()) // 2) / (n_layers * sh.top_k * max(1, steps - 1))
        us_tok = ms * 1e3 / steps
        t_link = nbytes / steps / (h2d_gbs * 1e9) * 1e6
        t_hbm = n_layers * sh.top_k * W.expert_bytes(sh) / (peaks()["hbm_gbs"] * 1e9) * 1e6
        runs.append({"trace": label, "target_exrep": target, "exrep": round(exrep, 4), "us_per_token": round(us_tok, 1),
                     "tokens_per_s": round(1e6 / us_tok, 2), "fetch_bytes_per_token": int(nbytes / steps),
                     "host_link_GB_per_s": round(nbytes / steps / (us_tok * 1e-6) / 1e9, 2),
                     "frac_of_floor": round(max(t_link, t_hbm) / us_tok, 4),
                     "host_wall_us_per_token": round(wall * 1e6 / steps, 1)})
    clocks = sampler.stop()
    main_run = runs[0]
    line = {
        "metric": "moe_stack_us_per_token_decode_offload_eq8", "value": main_run["us_per_token"], "unit": "us/token",
        "n_gpus": 1, "steps": steps, "warmup": 1, "ms_per_step": round(main_run["us_per_token"] / 1e3, 4),
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 weights/activations, f32 accumulate", "data": "synthetic",
        "config": {"workload": "phone-offload-eq8", "shape": W.describe(sh), "layers": n_layers,
                   "resident_slots_per_layer": sh.top_k, "T": 1,
                   "launch_mode": "stream (host queues a whole token, one sync per token)",
                   "l2": "inputs larger than L2: distinct layers per token"},
        "roofline": {"bound": "host_link", "achieved": main_run["host_link_GB_per_s"], "peak": round(h2d_gbs, 2),
                     "unit": "GB/s", "frac": main_run["frac_of_floor"], "traffic": None,
                     "peak_source": "pinned H2D copy of one expert, measured in this run"},
        "runs": runs,
        "speedup_from_stickier_routing": round(runs[0]["us_per_token"] / runs[1]["us_per_token"], 2),
        "e2e": {"value": main_run["host_wall_us_per_token"], "unit": "us/token",
                "h2d_bytes_per_step": main_run["fetch_bytes_per_token"], "d2h_bytes_per_step": 0},
        "gpu_launches": int(B.moe_launch_count(stack.ctx)),
        "clocks": clocks,
    }
    print(json.dumps(line))
    stack.close()
    return 0


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """A time measured on every rank -> the slowest rank's (all ranks get it).  Replicas exchange nothing else."""
    if world <= 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def aggregate(metric_kind: str, T: int, ms_per_step: float, world: int):
    """Whole-job value for `world` replicas that each ran the same steps in ms_per_step (max over ranks)."""
    return metric_of({"T": T, "kind": metric_kind}, ms_per_step, world)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4096)
    ap.add_argument("--warmup", type=int, default=64)
    ap.add_argument("--workload", default=DEFAULT, choices=sorted(WORKLOADS) + ["phone-offload-stack", "phone-offload-eq8"])
    ap.add_argument("--layers", type=int, default=24, help="phone-offload-stack: stacked layers")
    ap.add_argument("--slots", type=int, default=4, help="phone-offload-stack: resident experts per layer")
    ap.add_argument("--decode-steps", type=int, default=256, help="phone-offload-stack: tokens")
    ap.add_argument("--all", action="store_true", help="(default behaviour now; kept for old command lines)")
    ap.add_argument("--no-others", action="store_true", help="time the main workload only")
    ap.add_argument("--fp8-host", action="store_true", help="phone-offload-stack: host copies as FP8 codes + row scales")
    ap.add_argument("--others-offload-steps", type=int, default=32, help="tokens of the shortened offload stack in 'others'")
    ap.add_argument("--sweep", action="store_true", help="also time the shape sweep (reported under 'sweep')")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ring", type=int, default=0, help="override the number of distinct layers in the ring")
    ap.add_argument("--no-graph", action="store_true", help="plain stream launches instead of a CUDA graph")
    ap.add_argument("--min-ms", type=float, default=1500.0,
                    help="repeat the timed steps until the region is at least this long (0: exactly --steps, for profiling)")
    a = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    a.warmup = max(a.warmup, 3)

    if a.impl == "reference":
        if rank != 0:
            return 0
        shape, T, kind = WORKLOADS[a.workload]
        cb = cpu_baseline(a.workload, budget_s=min(60.0, 2.0 * max(1, a.steps // 512)))
        line = {"impl": "reference", "metric": metric_of({"T": T, "kind": kind}, 1.0)[0], "value": cb["value"],
                "unit": cb["unit"], "n_gpus": 0, "steps": a.steps, "warmup": a.warmup,
                "ms_per_step": cb["value"] * T / 1e3 if kind == "decode" else T / cb["value"] * 1e3,
                "higher_is_better": kind != "decode", "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic", "config": {"workload": a.workload, "shape": W.describe(shape), "T": T},
                "cpu_baseline": cb,
                "e2e": {"value": cb["value"], "unit": cb["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return 0

    if not torch.cuda.is_available():
        sys.stderr.write("bench.py: no CUDA device; the layer has no CPU fallback\n")
        return 2
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=device)
    from paper_2503_00245_b200 import build as _b
    if rank == 0:
        _b.build()
    if world > 1:
        torch.distributed.barrier()

    if a.workload == "phone-offload-stack":
        return run_offload_stack(a, device, fp8=a.fp8_host) if rank == 0 else 0
    if a.workload == "phone-offload-eq8":
        return run_offload_eq8(a, device) if rank == 0 else 0
    res = time_workload(a.workload, a.steps, a.warmup, device, rank, world, a.ring, not a.no_graph, a.min_ms)
    ms_per_step = max_over_ranks(res["ms_total"], world, device) / res["steps"]
    metric, value, unit, hib = metric_of(res, ms_per_step, world)
    e2e_ms, h2d, d2h = e2e_measure(res, a.steps)
    _, e2e_val, _, _ = metric_of(res, max_over_ranks(e2e_ms, world, device), world)

    others = []
    if not a.no_others and rank == 0 and world == 1 and a.workload == DEFAULT:
        res.pop("ring", None)
        torch.cuda.empty_cache()
        for name in OTHERS:
            try:
                r = time_workload(name, min(a.steps, 1024), a.warmup, device, rank, 1, min_ms=400.0)
            except Exception as e:  # noqa: BLE001
                others.append({"workload": name, "error": str(e)[:200]})
                continue
            m, v, u, _ = metric_of(r, r["ms_per_step"])
            others.append({"workload": name, "metric": m, "value": round(v, 3), "unit": u, "steps": r["steps"],
                           "ms_per_step": round(r["ms_per_step"], 5), "launch_mode": r["launch_mode"],
                           "launches_per_step": r["launches_per_step"],
                           "active_experts_per_step": r["active_experts_per_step"], "roofline": roofline(r),
                           "clocks": r["clocks"]})
            del r
            torch.cuda.empty_cache()
        saved = a.decode_steps
        a.decode_steps = a.others_offload_steps
        for fp8 in (False, True):
            name = "phone-offload-stack-fp8" if fp8 else "phone-offload-stack"
            try:
                o = run_offload_stack(a, device, emit=False, fp8=fp8)
                others.append({"workload": name, "metric": o["metric"], "value": o["value"], "unit": o["unit"],
                               "steps": o["steps"], "ms_per_step": o["ms_per_step"], "config": o["config"],
                               "roofline": o["roofline"], "offload": o["offload"], "clocks": o["clocks"]})
            except Exception as e:  # noqa: BLE001
                others.append({"workload": name, "error": str(e)[:200]})
        a.decode_steps = saved

    sweep = []
    if a.sweep and rank == 0 and world == 1:
        res.pop("ring", None)
        torch.cuda.empty_cache()
        for name in SWEEP:
            try:
                r = time_workload(name, min(a.steps, 1024), a.warmup, device, rank, 1)
            except Exception as e:  # noqa: BLE001
                sweep.append({"workload": name, "error": str(e)[:200]})
                continue
            rf = roofline(r)
            sweep.append({"workload": name, "shape": W.describe(r["shape"]), "us_per_token": round(r["ms_per_step"] * 1e3, 3),
                          "GB_per_s": rf["achieved"], "frac": rf["frac"]})
            del r
            torch.cuda.empty_cache()

    if rank == 0:
        shape, T = res["shape"], res["T"]
        line = {
            "metric": metric, "value": round(value, 4), "unit": unit, "n_gpus": world, "steps": res["steps"],
            "warmup": a.warmup, "ms_per_step": round(ms_per_step, 6), "higher_is_better": hib, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 weights/activations, f32 accumulate", "data": "synthetic",
            "config": {"workload": a.workload, "shape": W.describe(shape), "T": T,
                       "launch_mode": res["launch_mode"], "ring_layers": res["ring_layers"],
                       "l2": "inputs larger than L2: ring of distinct layers, touched weights >= 4x L2",
                       "active_experts_per_step": res["active_experts_per_step"],
                       "parallelism": "replicas only (no collective)" if world > 1 else "1 GPU"},
            "roofline": roofline(res),
            "e2e": {"value": round(e2e_val, 4), "unit": unit, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "how": "pinned x -> device copy, moe_layer_forward, y -> pinned host copy, stream wait, per step"},
            "gpu_launches": int(round(res["launches_per_step"] * res["steps"])),
            "clocks": res["clocks"],
        }
        if res.get("e2e_mapped_ms") is not None and world == 1:
            line["e2e"]["y_in_mapped_host_memory"] = {
                "value": round(metric_of(res, res["e2e_mapped_ms"])[1], 4), "unit": unit,
                "how": "pinned x -> device copy, moe_layer_forward with y in mapped pinned host memory, stream wait, per step"}
        if not a.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(a.workload)
        if others:
            line["others"] = others
        if sweep:
            line["sweep"] = sweep
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
