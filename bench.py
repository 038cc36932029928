#!/usr/bin/env python
"""Benchmark of the EntropyCache cached denoising step on B200 (libentropycache).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One *step* is one denoising step of the hot path over one batch of synthetic
input: for every layer `ec_attend` (scatter-refresh of the active rows' K/V, then
active-row bidirectional attention over the whole cache) followed by one
`ec_entropy_gate` over the block's logits.  The headline `value` is the time of
a SKIP step per layer (microseconds per layer-step: refresh + 34-row attention,
plus the gate amortised over the layers) on the full-depth configuration
(LLaDA geometry, L = 4096, 32 layers, batch 1: the largest single-GPU workload of
the benchmark); the same quantity for a RECOMPUTE step (every row active) is
reported beside it, as the metric asks ("skip vs recompute").  Layers use
distinct K/V caches whose total size exceeds the L2 cache several times, so
every layer-step streams its cache from HBM.  `per_workload` carries the same
measurements (shorter regions) for every other benchmark shape, each with its
three rooflines and the clocks sampled during its own region.

Timing: CUDA events on the launching stream around exactly K replays of a CUDA
graph that holds one whole step; W untimed warm-up replays first; max over ranks.
With N > 1 every rank runs the same per-GPU workload on its own sequences (the
path shards by sequence with no exchange): weak scaling, no data-path collective.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import ec_synth as syn  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
DEFAULT_WORKLOAD = "c5_llada_l4096"
# shapes reported in `per_workload` beside the headline one (the configurations of the benchmark, batch 1 and 8,
# both model geometries)
PER_WORKLOAD = ("c2_llada_l768", "c3_dream_l768", "c4_llada_l2048", "c5_llada_l4096", "c5_llada_l4096_b8",
                "c4_dream_l2048", "c5_dream_l4096")
K64_WORKLOADS = ("c4_llada_l2048", "c5_llada_l4096", "c5_llada_l4096_b8", "c5_dream_l4096")   # also timed at the paper's k = 64


# DRAM traffic per launch (reads + writes: dram__bytes.sum.per_second x gpu__time_duration.sum) from the ncu captures
# summarised under profiles/.  A figure is reported only while the kernel's source file still has the hash it had when the
# counters were taken; after any change to the kernel it reads null until the capture is redone.
NCU_TRAFFIC = {
    "attend_skip": [
        {"source": "paper_2603_18489_b200/csrc/ec_attend_skip_keys_tc.cu",
         "sha256": "55eea1c65c1cfe60b79f17c4d0f5c2d222cf29ddff308fb432c5a73e07d8b972",
         "bytes_per_launch": {"c2_llada_l768": 13400000, "c5_llada_l4096": 68730000}},
        {"source": "paper_2603_18489_b200/csrc/ec_attend_skip_tc.cu",
         "sha256": "bfec166c49fcaea673858dc2e86bfa2b1bffe4d191e2c41857dac13d2d180d5a",
         "bytes_per_launch": {"c5_llada_l4096_b8": 552480000}}],
    "attend_dense": [
        {"source": "paper_2603_18489_b200/csrc/ec_attend_dense_tc.cu",
         "sha256": "4323d044418277f0fa12a7dee721db22bf5b7291e5e7e0507861c74d0b3dd4fe",
         "bytes_per_launch": {"c2_llada_l768": 18930000, "c4_llada_l2048": 62770000, "c5_llada_l4096": 176240000}}],
    "entropy_gate": [
        {"source": "paper_2603_18489_b200/csrc/ec_gate.cu",
         "sha256": "519bc6a99b3932ab141af3aa77056dff693970d2254c54c7a023263874293215",
         "bytes_per_launch": {"c5_llada_l4096": 8140000, "c5_llada_l4096_b8": 65060000}}],
}


def _ncu_traffic(kernel: str, workload: str):
    import hashlib

    for e in NCU_TRAFFIC[kernel]:
        if workload not in e["bytes_per_launch"]:
            continue
        try:
            h = hashlib.sha256(open(os.path.join(ROOT, e["source"]), "rb").read()).hexdigest()
        except OSError:
            return None
        return e["bytes_per_launch"][workload] if h == e["sha256"] else None
    return None


def _peaks() -> dict:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# --------------------------------------------------------------------------- #
# clocks sampler
# --------------------------------------------------------------------------- #
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- #
# device-side workload
# --------------------------------------------------------------------------- #
class DeviceWorkload:
    """Synthetic tensors of one workload on one GPU: n_layers distinct K/V caches
    (seeded torch generator on the device; same value laws as ec_synth)."""

    def __init__(self, w: syn.Workload, n_layers: int, device, seed: int, need_recompute: bool = True,
                 need_gate: bool = True):
        import torch
        import paper_2603_18489_b200 as ec

        self.w, self.n_layers, self.ec, self.torch = w, n_layers, ec, torch
        g = torch.Generator(device=device)
        g.manual_seed(seed)
        dt = torch.bfloat16 if w.dtype == syn.BF16 else torch.float32
        B, L, Hq, Hkv, D = w.batch, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim
        std = 1.0 / np.sqrt(D)

        def rn(*shape):
            return (torch.randn(*shape, generator=g, device=device, dtype=torch.float32) * std).to(dt)

        # Consecutive launches of a step work on different layers' caches, so nothing in flight writes the caches a
        # launch reads: the bench states that (EC_ATTN_CACHE_SETTLED), as a model's layer loop would, whose attention
        # follows the projection that produced q / k_new / v_new.  With a single layer the statement would be false.
        self.desc_plain = ec.make_desc(B, L, Hq, Hkv, D, w.dtype)
        self.desc = ec.make_desc(B, L, Hq, Hkv, D, w.dtype,
                                 flags=ec.EC_ATTN_CACHE_SETTLED if n_layers >= 2 else 0)
        self.k_cache = [rn(B, Hkv, L, D) for _ in range(n_layers)]
        self.v_cache = [rn(B, Hkv, L, D) for _ in range(n_layers)]
        n = w.n_skip_rows
        self.n_skip = n
        self.q_s = [rn(B, n, Hq, D) for _ in range(n_layers)]
        self.kn_s = [rn(B, n, Hkv, D) for _ in range(n_layers)]
        self.vn_s = [rn(B, n, Hkv, D) for _ in range(n_layers)]
        self.out_s = [torch.empty(B, n, Hq, D, device=device, dtype=dt) for _ in range(n_layers)]
        idx = syn.active_rows(w, block_no=(w.gen_len // w.block) // 2)
        self.idx_np = idx
        self.idx = torch.from_numpy(idx).to(device)
        self.ws_s = ec.new_workspace(ec.ec_attend_workspace_bytes(self.desc, n), device)
        self.n_fresh = 0
        if need_recompute:
            # fresh tensors of the recompute step (every row active): enough distinct sets, used in rotation by the
            # layers, that a layer finds neither its q / k_new / v_new nor its cache in L2 (each layer owns its cache)
            set_bytes = (2 * Hq + 2 * Hkv) * B * L * D * syn.elem_bytes(w.dtype)   # q, out, k_new, v_new
            self.n_fresh = int(min(n_layers, max(1, np.ceil(2.5 * L2_BYTES / set_bytes))))
            self.q_r = [rn(B, L, Hq, D) for _ in range(self.n_fresh)]
            self.kn_r = [rn(B, L, Hkv, D) for _ in range(self.n_fresh)]
            self.vn_r = [rn(B, L, Hkv, D) for _ in range(self.n_fresh)]
            self.out_r = [torch.empty(B, L, Hq, D, device=device, dtype=dt) for _ in range(self.n_fresh)]
            self.ws_r = ec.new_workspace(ec.ec_attend_workspace_bytes(self.desc, L), device)
        # logits: rows ~ N(0, sigma_r^2), sigma_r ~ U(0.5, 8); several buffers so a gate-only loop is cold
        R = w.n_logit_rows
        self.R = R
        self.n_lbuf = 0
        if not need_gate:
            return
        n_lbuf = max(2, int(np.ceil(2.2 * L2_BYTES / (R * w.vocab * syn.elem_bytes(w.dtype)))))
        self.n_lbuf = min(n_lbuf, 40)
        self.logits = []
        for _ in range(self.n_lbuf):
            sig = torch.rand(R, 1, generator=g, device=device) * 7.5 + 0.5
            self.logits.append((torch.randn(R, w.vocab, generator=g, device=device) * sig).to(dt))
        fl = syn.decoded_flags(R, 16, w.block, cfg_id=w.cfg_id)
        self.flags_np = fl
        self.flags = torch.from_numpy(fl).to(device)
        self.ws_g = ec.new_workspace(ec.ec_entropy_gate_workspace_bytes(R, w.vocab), device)
        nseq = R // w.block
        self.maxh = torch.empty(nseq, device=device, dtype=torch.float32)
        self.dec = torch.empty(nseq, device=device, dtype=torch.int32)
        self.argmax = torch.empty(R, device=device, dtype=torch.int32)
        self.conf = torch.empty(R, device=device, dtype=torch.float32)
        self.ent = torch.empty(R, device=device, dtype=torch.float32)
        self.tau = 1.5
        self._gate_i = 0

    # -- single calls (asynchronous on the current stream) ------------------------
    def attend_skip(self, l: int, refresh: bool = True, settled: bool = True):
        self.ec.ec_attend(self.desc if settled else self.desc_plain, self.q_s[l], self.kn_s[l] if refresh else None,
                          self.vn_s[l] if refresh else None, self.k_cache[l], self.v_cache[l], self.idx,
                          out=self.out_s[l], workspace=self.ws_s)

    def attend_recompute(self, l: int, refresh: bool = True):
        f = l % self.n_fresh
        self.ec.ec_attend(self.desc, self.q_r[f], self.kn_r[f] if refresh else None, self.vn_r[f] if refresh else None,
                          self.k_cache[l], self.v_cache[l], None, out=self.out_r[f], workspace=self.ws_r)

    def kernel_names(self) -> dict:
        """The launches the library makes for this workload's skip and recompute steps (host-only query)."""
        return {"skip": self.ec.ec_attend_kernel_name(self.desc, self.n_skip, True, True),
                "recompute": self.ec.ec_attend_kernel_name(self.desc, self.w.ctx_len, True, False)}

    def gate(self, i: int | None = None):
        if i is None:
            i = self._gate_i
            self._gate_i = (self._gate_i + 1) % self.n_lbuf
        self.ec.ec_entropy_gate(self.logits[i], self.w.vocab, self.w.block, self.flags, self.tau,
                                argmax_out=self.argmax, conf_out=self.conf, entropy_out=self.ent,
                                max_entropy_out=self.maxh, decision_out=self.dec, workspace=self.ws_g)

    # -- algorithmic bytes / flops (per layer-step and per gate call) --------------
    def skip_bytes(self) -> int:
        w, s, n = self.w, syn.elem_bytes(self.w.dtype), self.n_skip
        per_seq = (2 * w.ctx_len * w.n_kv_heads * w.head_dim * s + 4 * n * w.n_kv_heads * w.head_dim * s
                   + 2 * n * w.n_q_heads * w.head_dim * s + 4 * n)
        return per_seq * w.batch

    def recompute_flops(self) -> int:
        w = self.w
        return 4 * w.ctx_len * w.ctx_len * w.head_dim * w.n_q_heads * w.batch

    def gate_bytes(self) -> int:
        return self.R * self.w.vocab * syn.elem_bytes(self.w.dtype) + 12 * self.R


def max_over_ranks(ms: float, dist, device) -> float:
    """The step time of the whole job is the slowest rank's (replicas: no other exchange between ranks)."""
    if dist is None:
        return ms
    import torch

    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def _graph_time(torch, body, replays: int, warmup: int, stream) -> float:
    """Captures body() into a CUDA graph, replays it `warmup` times untimed and `replays`
    times timed; returns milliseconds per replay (CUDA events on the launching stream)."""
    with torch.cuda.stream(stream):
        body()  # eager once: first-call set-up (function attributes) must not happen under capture
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            body()
        for _ in range(warmup):
            g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(replays):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) / replays


def _workload(args) -> syn.Workload:
    """The named workload, with the recent-token budget replaced when --k-recent is given (the paper's default is
    k = 64 and its grid 16..256; the named workloads use 2)."""
    import dataclasses

    w = syn.WORKLOADS[args.workload]
    if getattr(args, "k_recent", -1) >= 0:
        w = dataclasses.replace(w, k_recent=args.k_recent)
    return w


def _choose_layers(w: syn.Workload) -> int:
    """Distinct K/V caches per step: the workload's own depth where it names one and it fits comfortably (the
    full-depth configuration at batch 1: 32 layers, 2 GiB), otherwise enough that a step streams 3x the L2."""
    per_layer = 2 * w.batch * w.ctx_len * w.n_kv_heads * w.head_dim * syn.elem_bytes(w.dtype)
    need = int(min(max(int(np.ceil(3.0 * L2_BYTES / per_layer)), 4), 64))
    if w.n_layers > need and w.n_layers * per_layer <= 4 << 30:
        return w.n_layers
    return need


def _config(w: syn.Workload, n_layers: int) -> dict:
    """The `config` object of the JSON line, the same for the CUDA arm and the reference arm."""
    kv_mib = n_layers * 2 * w.batch * w.ctx_len * w.n_kv_heads * w.head_dim * syn.elem_bytes(w.dtype) >> 20
    return {"workload": w.name, "n_layers": n_layers, "batch": w.batch, "ctx_len": w.ctx_len,
            "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
            "n_active_skip": w.n_skip_rows, "vocab": w.vocab, "logit_rows": w.n_logit_rows,
            "desc_flags": "EC_ATTN_CACHE_SETTLED" if n_layers >= 2 else "0",
            "l2": f"inputs larger than L2: {n_layers} distinct K/V caches ({kv_mib} MiB) per step; the recompute "
                  f"step's fresh q/k/v rotate over sets that together exceed 2.5x L2; logits rotate over buffers "
                  f"that exceed 2.2x L2"}


# --------------------------------------------------------------------------- #
# CPU oracle legs
# --------------------------------------------------------------------------- #
_ORACLE_INPUTS: dict = {}


def _oracle_inputs(w: syn.Workload):
    """Seeded host tensors of one skip layer-step and one gate call (drawn once per workload and process)."""
    if w.name not in _ORACLE_INPUTS:
        t = syn.attn_inputs(w, w.n_skip_rows)
        lg = syn.logits_rows(w.n_logit_rows, w.vocab, w.dtype, cfg_id=w.cfg_id)
        fl = syn.decoded_flags(w.n_logit_rows, 16, w.block, cfg_id=w.cfg_id)
        _ORACLE_INPUTS[w.name] = (t, lg, fl)
    return _ORACLE_INPUTS[w.name]


def _oracle_layer_step_us(w: syn.Workload, reps: int = 1) -> dict:
    """Times the oracle (as it stands) on one skip layer-step and one gate call of workload w."""
    import oracle

    t, lg, fl = _oracle_inputs(w)
    oracle.entropy_gate(lg["logits"][:1], w.dtype, w.vocab, fl[:1], 1.5, 1)  # load + warm the library
    ta, tg = [], []
    for _ in range(reps):
        kc, vc = t["k_cache"].copy(), t["v_cache"].copy()
        t0 = time.perf_counter()
        oracle.refresh_and_attend(t["q"], t["k_new"], t["v_new"], kc, vc, t["active_idx"], w.dtype)
        t1 = time.perf_counter()
        oracle.entropy_gate(lg["logits"], w.dtype, w.vocab, fl, 1.5, w.block)
        t2 = time.perf_counter()
        ta.append(t1 - t0)
        tg.append(t2 - t1)
    return dict(attend_us=min(ta) * 1e6, gate_us=min(tg) * 1e6, cores=oracle.num_threads())


def run_reference(args) -> None:
    """The reference arm: the oracle as it stands on the host cores.  One step = one skip layer-step (refresh +
    active-row attention over the whole cache of ONE layer) and one gate call: a bounded sample of the CUDA arm's step
    (which runs n_layers layer-steps); `value` is the same metric (layer-step + the gate amortised over the layers),
    `ms_per_step` the time the sample really took."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = _workload(args)
    n_layers = args.layers or _choose_layers(w)
    for _ in range(args.warmup):
        _oracle_layer_step_us(w, 1)
    vals, walls = [], []
    cores = 1
    for _ in range(args.steps):
        r = _oracle_layer_step_us(w, 1)
        cores = r["cores"]
        vals.append(r["attend_us"] + r["gate_us"] / n_layers)
        walls.append(r["attend_us"] + r["gate_us"])
    v = float(np.mean(vals))
    sample = (f"per step: 1 of the {n_layers} skip layer-steps (refresh + {w.n_skip_rows}-row attention over "
              f"L={w.ctx_len}) + 1 gate call [{w.n_logit_rows}x{w.vocab}]; value = layer-step + gate / {n_layers}")
    line = {
        "impl": "reference", "metric": "us_per_layer_step_skip", "value": v, "unit": "us", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(walls)) / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config(w, n_layers),
        "cpu_baseline": {"value": v, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- #
# main arm
# --------------------------------------------------------------------------- #
def _rooflines(wl: "DeviceWorkload", peaks: dict, ms_skip_launch: float, ms_rec_launch: float, ms_gate: float) -> dict:
    """The three roofline objects of a workload from the average launch durations (milliseconds) of its regions.
    Units of one launch: skip = one layer-step of the whole batch (refresh + attention + merge: skip_bytes),
    recompute = one layer-step (recompute_flops; its refresh copy rides in the same launch), gate = R rows."""
    w = wl.w
    skip_b, rec_f, gate_b = wl.skip_bytes(), wl.recompute_flops(), wl.gate_bytes()
    att_gbs = skip_b / (ms_skip_launch * 1e-3) / 1e9
    rec_tf = rec_f / (ms_rec_launch * 1e-3) / 1e12
    gate_gbs = gate_b / (ms_gate * 1e-3) / 1e9
    return {
        "roofline": {"kernel": "ec_attend skip step (one launch: refresh + attention + merge)", "bound": "hbm",
                     "achieved": att_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": att_gbs / peaks["hbm_gbs"],
                     "traffic": _ncu_traffic("attend_skip", w.name), "algorithmic_bytes": skip_b,
                     "us_per_launch": ms_skip_launch * 1e3, "peak_source": peaks["source"]},
        "roofline_recompute": {"kernel": "ec_attend recompute step (one launch: attention + cache rewrite)",
                               "bound": "tensor", "achieved": rec_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                               "frac": rec_tf / peaks["bf16_tflops"], "traffic": _ncu_traffic("attend_dense", w.name),
                               "algorithmic_flops": rec_f, "us_per_launch": ms_rec_launch * 1e3,
                               "peak_source": peaks["source"] + " (burst: the kernel is timed alone)"},
        "roofline_gate": {"kernel": "ec_entropy_gate", "bound": "hbm", "achieved": gate_gbs, "peak": peaks["hbm_gbs"],
                          "unit": "GB/s", "frac": gate_gbs / peaks["hbm_gbs"],
                          "traffic": _ncu_traffic("entropy_gate", w.name), "algorithmic_bytes": gate_b,
                          "us_per_launch": ms_gate * 1e3, "peak_source": peaks["source"]},
    }


def _measure_workload(torch, w: syn.Workload, n_layers: int, dev, stream, peaks: dict, reps: int, seed: int,
                      local_gpu: int, sample_clocks: bool) -> dict:
    """Per-kernel regions of one workload, each its own CUDA graph timed with CUDA events on the launching stream:
    skip layer-steps (refresh inside the launch), recompute layer-steps, gate calls over rotating logits buffers."""
    wl = DeviceWorkload(w, n_layers, dev, seed=seed)
    sampler = ClockSampler(local_gpu) if sample_clocks else None
    if sampler:
        sampler.start()
        time.sleep(0.15)
    ms_skip = _graph_time(torch, lambda: [wl.attend_skip(l) for l in range(n_layers)], reps, 3, stream) / n_layers
    ms_gate = _graph_time(torch, lambda: [wl.gate(i) for i in range(wl.n_lbuf)], reps, 3, stream) / wl.n_lbuf
    # the dense region last: its power draw lowers the clocks for what follows
    ms_rec = _graph_time(torch, lambda: [wl.attend_recompute(l) for l in range(n_layers)], reps, 3, stream) / n_layers
    clocks = sampler.stop() if sampler else None
    out = {"n_layers": n_layers, "batch": w.batch, "ctx_len": w.ctx_len, "n_active_skip": wl.n_skip,
           "kernels": wl.kernel_names(),
           "us_per_layer_step": {"skip": ms_skip * 1e3 + ms_gate * 1e3 / n_layers,
                                 "recompute": ms_rec * 1e3 + ms_gate * 1e3 / n_layers},
           "clocks": clocks}
    out.update(_rooflines(wl, peaks, ms_skip, ms_rec, ms_gate))
    return out


def _measure_k64(torch, w: syn.Workload, n_layers: int, dev, stream, peaks: dict, reps: int, seed: int) -> dict:
    """The skip layer-step at the paper's default budget k = 64 (96 active rows): same caches' shape, same timing."""
    import dataclasses

    w64 = dataclasses.replace(w, k_recent=64)
    wl = DeviceWorkload(w64, n_layers, dev, seed=seed, need_recompute=False, need_gate=False)
    ms = _graph_time(torch, lambda: [wl.attend_skip(l) for l in range(n_layers)], reps, 3, stream) / n_layers
    gbs = wl.skip_bytes() / (ms * 1e-3) / 1e9
    return {"n_active_skip": wl.n_skip, "kernel": wl.kernel_names()["skip"], "us_per_launch": ms * 1e3,
            "algorithmic_bytes": wl.skip_bytes(), "achieved": gbs, "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"]}


def run_cuda(args) -> None:
    import gc

    import torch
    import paper_2603_18489_b200 as ec  # raises if the CUDA library is not built: no fallback

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_

        dist = dist_
        dist.init_process_group("nccl", device_id=dev)

    w = _workload(args)
    n_layers = args.layers or _choose_layers(w)
    peaks = _peaks()
    if args.trace:
        (_run_trace_sliding if args.sliding else _run_trace)(args, torch, w, dev)
        return
    if args.only:
        _run_only(args, torch, w, n_layers, dev)
        return
    wl = DeviceWorkload(w, n_layers, dev, seed=1234 + rank)
    stream = torch.cuda.Stream(device=dev)
    K, W = args.steps, max(args.warmup, 3)

    def skip_step():
        for l in range(n_layers):
            wl.attend_skip(l)
        wl.gate()

    def recompute_step():
        for l in range(n_layers):
            wl.attend_recompute(l)
        wl.gate()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_max(ms: float) -> float:
        return max_over_ranks(ms, dist, dev)

    # ---- headline: K skip steps, then K recompute steps ----------------------------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    ms_skip = reduce_max(_graph_time(torch, skip_step, K, W, stream))
    barrier()
    # ---- per-kernel regions for the rooflines (rank-local, same buffers, same stream, same clock record) ----
    # the skip region times the launch the algorithmic bytes describe: refresh + attention + merge in one kernel.
    # The two HBM-bound regions run before the dense ones, whose power draw lowers the clocks for what follows.
    reps = max(K, 5)
    ms_att_skip = _graph_time(torch, lambda: [wl.attend_skip(l) for l in range(n_layers)], reps, 3, stream) / n_layers
    ms_gate = _graph_time(torch, lambda: [wl.gate(i) for i in range(wl.n_lbuf)], reps, 3, stream) / wl.n_lbuf
    barrier()
    ms_rec = reduce_max(_graph_time(torch, recompute_step, K, W, stream))
    barrier()
    ms_att_rec = _graph_time(torch, lambda: [wl.attend_recompute(l) for l in range(n_layers)], reps, 3, stream) / n_layers
    clocks = sampler.stop() if rank == 0 else None
    ms_att_only = _graph_time(torch, lambda: [wl.attend_skip(l, refresh=False) for l in range(n_layers)], reps, 3,
                              stream) / n_layers
    ms_att_serial = _graph_time(torch, lambda: [wl.attend_skip(l, settled=False) for l in range(n_layers)], reps, 3,
                                stream) / n_layers
    ms_refresh = _graph_time(
        torch, lambda: [ec.ec_kv_refresh(wl.desc, wl.k_cache[l], wl.v_cache[l], wl.kn_s[l], wl.vn_s[l], wl.idx)
                        for l in range(n_layers)], reps, 3, stream) / n_layers

    # the loop's bookkeeping on the device (decode history, recent set, next row list): eight calls per replay
    sel_hist, sel_state = ec.new_history(w.batch, w.ctx_len, dev), ec.new_step_state(w.batch, 1, dev)
    sel_idx = torch.empty(w.batch, w.block + 64, dtype=torch.int32, device=dev)
    sel_w0 = torch.full((w.batch,), w.prompt_len, dtype=torch.int32, device=dev)

    def select_only():
        for _ in range(8):
            ec.ec_select_recent(sel_hist, sel_state, wl.flags, sel_w0, w.block, wl.dec, w.k_recent, sel_idx)

    ms_select = _graph_time(torch, select_only, reps, 3, stream) / 8

    ms_e2e, h2d, d2h = _e2e(torch, ec, wl, w, n_layers, dev, stream, K, barrier)
    ms_e2e = reduce_max(ms_e2e)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    us_skip = ms_skip * 1e3 / n_layers / world
    us_rec = ms_rec * 1e3 / n_layers / world
    cpu = _oracle_layer_step_us(w, 2)
    cfg = _config(w, n_layers)
    line = {
        "metric": "us_per_layer_step_skip", "value": us_skip, "unit": "us", "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms_skip, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.dtype == syn.BF16 else "f32", "data": "synthetic",
        "config": cfg,
        "timing": "one CUDA graph per step, CUDA events on the launching stream, max over ranks",
        "kernels": wl.kernel_names(),
        "recompute": {"us_per_layer_step": us_rec, "ms_per_step": ms_rec,
                      "skip_over_recompute": us_skip / us_rec},
        "kernels_us": {"attend_skip": ms_att_skip * 1e3, "attend_skip_without_refresh": ms_att_only * 1e3,
                       "attend_skip_without_cache_settled_flag": ms_att_serial * 1e3,
                       "attend_recompute": ms_att_rec * 1e3, "entropy_gate": ms_gate * 1e3,
                       "kv_refresh_skip": ms_refresh * 1e3, "select_recent": ms_select * 1e3},
        "e2e": {"value": ms_e2e * 1e3 / n_layers / world, "unit": "us", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": K * (n_layers + 1),   # a skip layer-step is one launch (refresh + attention + merge), + the gate
        "clocks": clocks,
    }
    line.update(_rooflines(wl, peaks, ms_att_skip, ms_att_rec, ms_gate))
    v = cpu["attend_us"] + cpu["gate_us"] / n_layers
    line["cpu_baseline"] = {
        "value": v, "unit": "us", "cores": cpu["cores"], "kind": "oracle",
        "sample": f"1 skip layer-step ({wl.n_skip} rows over L={w.ctx_len}, {cpu['attend_us']:.0f} us) + 1 gate "
                  f"call [{wl.R}x{w.vocab}] ({cpu['gate_us']:.0f} us) amortised over {n_layers} layers; best of 2"}

    # ---- the other benchmark shapes, same measurements over shorter regions (single GPU runs only) ----
    if world == 1 and not args.no_per_workload:
        del wl
        per = {}
        for name in PER_WORKLOAD:
            gc.collect()
            torch.cuda.empty_cache()
            wo = syn.WORKLOADS[name]
            nl = _choose_layers(wo)
            per[name] = _measure_workload(torch, wo, nl, dev, stream, peaks, 5, 1234, local, True)
            if name in K64_WORKLOADS:
                gc.collect()
                torch.cuda.empty_cache()
                per[name]["k64"] = _measure_k64(torch, wo, nl, dev, stream, peaks, 5, 1234)
        line["per_workload"] = per
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def _e2e(torch, ec, wl, w, n_layers: int, dev, stream, K: int, barrier):
    """End to end through the binding with host buffers: returns (ms per step, h2d bytes, d2h bytes).
    Per step every layer's q / k_new / v_new come from pinned host memory and every layer's output goes back, as do
    the step's logits and the gate's decision.  The layers' inputs sit back to back in one host arena and one device
    arena (the tensors the library sees are views), so a group of layers moves with ONE copy; inputs go up on one
    copy stream, results come back on another, the kernels run on the compute stream, and events order a group's
    kernels after its inputs and its read-back after its kernels: PCIe traffic in both directions overlaps the
    kernels of the neighbouring groups."""
    dt = torch.bfloat16 if w.dtype == syn.BF16 else torch.float32
    nq, nkv = wl.q_s[0].numel(), wl.kn_s[0].numel()
    per_layer = nq + 2 * nkv
    in_dev = torch.empty(n_layers * per_layer, device=dev, dtype=dt)
    in_host = torch.empty(n_layers * per_layer, dtype=dt).pin_memory()
    out_dev = torch.empty(n_layers * nq, device=dev, dtype=dt)
    out_host = torch.empty(n_layers * nq, dtype=dt).pin_memory()
    q_e, k_e, v_e, o_e = [], [], [], []
    for l in range(n_layers):
        o = l * per_layer
        q_e.append(in_dev[o:o + nq].view(wl.q_s[l].shape))
        k_e.append(in_dev[o + nq:o + nq + nkv].view(wl.kn_s[l].shape))
        v_e.append(in_dev[o + nq + nkv:o + per_layer].view(wl.vn_s[l].shape))
        o_e.append(out_dev[l * nq:(l + 1) * nq].view(wl.q_s[l].shape))
        in_host[o:o + nq].copy_(wl.q_s[l].reshape(-1).cpu())
        in_host[o + nq:o + nq + nkv].copy_(wl.kn_s[l].reshape(-1).cpu())
        in_host[o + nq + nkv:o + per_layer].copy_(wl.vn_s[l].reshape(-1).cpu())
    hlog = wl.logits[0].cpu().pin_memory()
    hdec = torch.empty_like(wl.dec, device="cpu").pin_memory()
    h2d = in_host.numel() * in_host.element_size() + hlog.numel() * hlog.element_size()
    d2h = out_host.numel() * out_host.element_size() + hdec.numel() * hdec.element_size()
    group = 4 if n_layers >= 8 else 1
    groups = [(g0, min(n_layers, g0 + group)) for g0 in range(0, n_layers, group)]
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(len(groups) + 1)]
    ev_done = [torch.cuda.Event() for _ in range(len(groups) + 1)]

    def e2e_step():
        with torch.cuda.stream(s_in):
            for gi, (l0, l1) in enumerate(groups):
                in_dev[l0 * per_layer:l1 * per_layer].copy_(in_host[l0 * per_layer:l1 * per_layer], non_blocking=True)
                ev_in[gi].record(s_in)
            wl.logits[0].copy_(hlog, non_blocking=True)
            ev_in[-1].record(s_in)
        for gi, (l0, l1) in enumerate(groups):
            stream.wait_event(ev_in[gi])
            with torch.cuda.stream(stream):
                for l in range(l0, l1):
                    ec.ec_attend(wl.desc, q_e[l], k_e[l], v_e[l], wl.k_cache[l], wl.v_cache[l], wl.idx, out=o_e[l],
                                 workspace=wl.ws_s)
            ev_done[gi].record(stream)
            s_out.wait_event(ev_done[gi])
            with torch.cuda.stream(s_out):
                out_host[l0 * nq:l1 * nq].copy_(out_dev[l0 * nq:l1 * nq], non_blocking=True)
        stream.wait_event(ev_in[-1])
        with torch.cuda.stream(stream):
            wl.gate(0)
        ev_done[-1].record(stream)
        s_out.wait_event(ev_done[-1])
        with torch.cuda.stream(s_out):
            hdec.copy_(wl.dec, non_blocking=True)
        s_out.synchronize()   # the host reads the decision to choose the next step's path ...
        stream.synchronize()  # ... and every stream is idle before the next step reuses the buffers
        s_in.synchronize()

    for _ in range(3):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(K):
        e2e_step()
    e1.record(stream)
    stream.synchronize()
    return e0.elapsed_time(e1) / K, h2d, d2h


def _run_trace(args, torch, w, dev) -> None:
    """Full-depth step trace (the fifth benchmark configuration): n_layers layers, every sequence of the batch
    with its own skip / recompute decision taken by ec_entropy_gate on that step's logits, the host reading
    the decisions back every step as the generation loop does (Algorithm 1).  Logits are seeded Gaussian rows
    whose sigma band drifts from step to step (a different phase per sequence); tau is set from a gate-only
    pre-pass so that about 15 % of the sequence-steps recompute (the paper's recompute ratios are 0.11-0.18).
    Prints one JSON line: time per step by kind and the skip / recompute cost per layer-step and sequence."""
    import paper_2603_18489_b200 as ec

    B, L, Hq, Hkv, D, V = w.batch, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.vocab
    n_layers = args.layers or w.n_layers
    n_steps = args.trace_steps or (w.n_steps if w.n_steps > 1 else 16)
    dt = torch.bfloat16 if w.dtype == syn.BF16 else torch.float32
    g = torch.Generator(device=dev)
    g.manual_seed(4321)
    std = 1.0 / np.sqrt(D)

    def rn(*shape):
        return (torch.randn(*shape, generator=g, device=dev, dtype=torch.float32) * std).to(dt)

    kc = [rn(B, Hkv, L, D) for _ in range(n_layers)]
    vc = [rn(B, Hkv, L, D) for _ in range(n_layers)]
    n = w.n_skip_rows
    q_s, kn_s, vn_s = rn(B, n, Hq, D), rn(B, n, Hkv, D), rn(B, n, Hkv, D)
    q_r, kn_r, vn_r = rn(B, L, Hq, D), rn(B, L, Hkv, D), rn(B, L, Hkv, D)
    out_s, out_r = torch.empty_like(q_s), torch.empty_like(q_r)
    idx = torch.from_numpy(syn.active_rows(w, block_no=(w.gen_len // w.block) // 2)).to(dev)
    d1 = ec.make_desc(1, L, Hq, Hkv, D, w.dtype)
    dB = ec.make_desc(B, L, Hq, Hkv, D, w.dtype)
    ws = ec.new_workspace(max(ec.ec_attend_workspace_bytes(dB, n), ec.ec_attend_workspace_bytes(dB, L)), dev)
    R = B * w.block
    period = 16
    logits = []
    for s_ in range(period):
        rows = []
        for b in range(B):
            centre = syn.drifting_sigma_centre(s_ + 2 * b, period)
            sig = torch.rand(w.block, 1, generator=g, device=dev) * 3.0 + max(0.25, centre - 1.5)
            rows.append((torch.randn(w.block, V, generator=g, device=dev) * sig).to(dt))
        logits.append(torch.cat(rows, 0))
    flags = torch.from_numpy(syn.decoded_flags(R, 4, w.block, cfg_id=w.cfg_id)).to(dev)
    ws_g = ec.new_workspace(ec.ec_entropy_gate_workspace_bytes(R, V), dev)
    maxh = torch.empty(B, device=dev, dtype=torch.float32)
    dec = torch.empty(B, device=dev, dtype=torch.int32)
    # tau from a gate-only pre-pass: the 85th percentile of the per-(step, sequence) maximum entropies
    E = []
    for lg in logits:
        ec.ec_entropy_gate(lg, V, w.block, flags, 0.0, max_entropy_out=maxh, decision_out=dec, workspace=ws_g,
                           want_rows=False)
        E.append(maxh.cpu().numpy().copy())
    tau = float(np.quantile(np.concatenate(E), 0.85))

    def attend(group, full: bool, layer: int):
        """One ec_attend per maximal run of consecutive sequences of the group."""
        for b0, nb in syn.consecutive_runs(group):
            d = ec.make_desc(nb, L, Hq, Hkv, D, w.dtype)
            sl = slice(b0, b0 + nb)
            if full:
                ec.ec_attend(d, q_r[sl], kn_r[sl], vn_r[sl], kc[layer][sl], vc[layer][sl], None, out=out_r[sl],
                             workspace=ws)
            else:
                ec.ec_attend(d, q_s[sl], kn_s[sl], vn_s[sl], kc[layer][sl], vc[layer][sl], idx[sl], out=out_s[sl],
                             workspace=ws)
        return len(syn.consecutive_runs(group))

    ev = lambda: torch.cuda.Event(enable_timing=True)
    decisions = np.ones(B, np.int64)   # step 1 is a full pass for every sequence
    t_skip = t_rec = t_gate = 0.0
    n_skip = n_rec = launches = 0
    per_step = []
    torch.cuda.synchronize()
    for s_ in range(n_steps):
        sk = [b for b in range(B) if decisions[b] == 0]
        rc = [b for b in range(B) if decisions[b] != 0]
        e0, e1, e2, e3 = ev(), ev(), ev(), ev()
        e0.record()
        for l in range(n_layers):
            launches += attend(sk, False, l)
        e1.record()
        for l in range(n_layers):
            launches += attend(rc, True, l)
        e2.record()
        ec.ec_entropy_gate(logits[s_ % period], V, w.block, flags, tau, max_entropy_out=maxh, decision_out=dec,
                           workspace=ws_g, want_rows=False)
        e3.record()
        decisions = dec.cpu().numpy().astype(np.int64)   # the host reads the decisions: they shape the next step
        launches += 1
        a, b_, c = e0.elapsed_time(e1) * 1e3, e1.elapsed_time(e2) * 1e3, e2.elapsed_time(e3) * 1e3
        if s_ > 0:   # the all-recompute first step warms everything up and is reported apart
            t_skip += a; t_rec += b_; t_gate += c
            n_skip += len(sk); n_rec += len(rc)
        per_step.append(dict(step=s_, n_skip=len(sk), n_recompute=len(rc), us=a + b_ + c))
    us_skip = t_skip / max(n_skip * n_layers, 1)
    us_rec = t_rec / max(n_rec * n_layers, 1)
    print(json.dumps({
        "trace": w.name, "n_layers": n_layers, "n_steps": n_steps, "batch": B, "tau": tau,
        "recompute_fraction": n_rec / max(n_skip + n_rec, 1),
        "us_per_layer_step_sequence": {"skip": us_skip, "recompute": us_rec},
        "skip_over_recompute": us_skip / us_rec if us_rec > 0 else None,
        "us_per_step_mean": {"attend_skip": t_skip / max(n_steps - 1, 1), "attend_recompute": t_rec / max(n_steps - 1, 1),
                             "gate": t_gate / max(n_steps - 1, 1)},
        "first_step_us": per_step[0]["us"], "gpu_launches": launches,
        "pattern": "".join("R" if p_["n_recompute"] == B else ("s" if p_["n_recompute"] == 0 else "m") for p_ in per_step),
        "timing": "CUDA events per step on the current stream, plain launches, host reads the decisions every step"}))


def _run_trace_sliding(args, torch, w, dev) -> None:
    """Step trace in the paper's own decoding mode (Section 2.1 / 5.1: a sliding window that keeps `window` mask
    tokens being denoised; its appendix varies the window from 8 to 128) with the whole loop state on the device:
    ec_entropy_gate_decode forms the decoded set from the confidences (threshold 0.9) and takes the gate's decision,
    ec_select_recent_sliding updates history, mask, recent set and writes the next row list, ec_attend takes that
    list from device memory (padded with -1 up to a fixed capacity).  The host reads one word per sequence and step
    (skip_flag, with the row count beside it) to pick the branch.  Prints one JSON line."""
    import paper_2603_18489_b200 as ec

    B, L, Hq, Hkv, D, V = w.batch, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.vocab
    window, k = args.window, w.k_recent
    n_layers = args.layers or _choose_layers(w)
    n_steps = args.trace_steps or (w.n_steps if w.n_steps > 1 else 16)
    n_cap = window + k + 8                      # ties at tau_R can add a few rows beyond k
    dt = torch.bfloat16 if w.dtype == syn.BF16 else torch.float32
    g = torch.Generator(device=dev)
    g.manual_seed(4321)
    std = 1.0 / np.sqrt(D)

    def rn(*shape):
        return (torch.randn(*shape, generator=g, device=dev, dtype=torch.float32) * std).to(dt)

    kc = [rn(B, Hkv, L, D) for _ in range(n_layers)]
    vc = [rn(B, Hkv, L, D) for _ in range(n_layers)]
    q_s, kn_s, vn_s = rn(B, n_cap, Hq, D), rn(B, n_cap, Hkv, D), rn(B, n_cap, Hkv, D)
    q_r, kn_r, vn_r = rn(B, L, Hq, D), rn(B, L, Hkv, D), rn(B, L, Hkv, D)
    out_s, out_r = torch.empty_like(q_s), torch.empty_like(q_r)
    ws = ec.new_workspace(max(ec.ec_attend_workspace_bytes(ec.make_desc(B, L, Hq, Hkv, D, w.dtype), n_cap),
                              ec.ec_attend_workspace_bytes(ec.make_desc(B, L, Hq, Hkv, D, w.dtype), L)), dev)
    R = B * window
    period = 16
    logits = []
    for s_ in range(period):
        rows = []
        for b in range(B):
            centre = syn.drifting_sigma_centre(s_ + 2 * b, period)
            sig = torch.rand(window, 1, generator=g, device=dev) * 3.0 + max(0.25, centre - 1.5)
            rows.append((torch.randn(window, V, generator=g, device=dev) * sig).to(dt))
        logits.append(torch.cat(rows, 0))
    ws_g = ec.new_workspace(ec.ec_entropy_gate_workspace_bytes(R, V), dev)
    maxh = torch.empty(B, device=dev, dtype=torch.float32)
    dec = torch.empty(B, device=dev, dtype=torch.int32)
    decoded = torch.empty(R, device=dev, dtype=torch.uint8)
    tokens = torch.full((R,), -1, device=dev, dtype=torch.int32)
    row_mask = torch.ones(R, device=dev, dtype=torch.uint8)      # every window row is a mask token, each step anew
    # tau: the 85th percentile of the per-(step, sequence) maximum entropies of a gate-only pre-pass
    E = []
    for lg in logits:
        row_mask.fill_(1)
        ec.ec_entropy_gate_decode(lg, V, window, row_mask, 0.9, 0.0, tokens, decoded_out=decoded, max_entropy_out=maxh,
                                  decision_out=dec, workspace=ws_g, want_rows=False)
        E.append(maxh.cpu().numpy().copy())
    tau = float(np.quantile(np.concatenate(E), 0.85))

    hist, state = ec.new_history(B, L, dev), ec.new_step_state(B, 1, dev)
    masked = torch.zeros(B, L, device=dev, dtype=torch.uint8)
    masked[:, w.prompt_len:] = 1
    idx = torch.full((B, n_cap), -1, device=dev, dtype=torch.int32)
    idx[:, :window] = torch.arange(w.prompt_len, w.prompt_len + window, device=dev, dtype=torch.int32)
    state_host = torch.empty(B, 4, dtype=torch.int32).pin_memory()

    ev = lambda: torch.cuda.Event(enable_timing=True)
    skip = np.zeros(B, bool)                    # step 1 is a full pass for every sequence
    t_skip = t_rec = t_book = 0.0
    n_skip = n_rec = launches = over_cap = 0
    per_step = []
    torch.cuda.synchronize()
    for s_ in range(n_steps):
        sk = [b for b in range(B) if skip[b]]
        rc = [b for b in range(B) if not skip[b]]
        e0, e1, e2, e3 = ev(), ev(), ev(), ev()
        e0.record()
        for l in range(n_layers):
            for b0, nb in syn.consecutive_runs(sk):
                sl = slice(b0, b0 + nb)
                ec.ec_attend(ec.make_desc(nb, L, Hq, Hkv, D, w.dtype), q_s[sl], kn_s[sl], vn_s[sl], kc[l][sl], vc[l][sl],
                             idx[sl], out=out_s[sl], workspace=ws)
                launches += 1
        e1.record()
        for l in range(n_layers):
            for b0, nb in syn.consecutive_runs(rc):
                sl = slice(b0, b0 + nb)
                ec.ec_attend(ec.make_desc(nb, L, Hq, Hkv, D, w.dtype), q_r[sl], kn_r[sl], vn_r[sl], kc[l][sl], vc[l][sl],
                             None, out=out_r[sl], workspace=ws)
                launches += 1
        e2.record()
        row_mask.fill_(1)
        ec.ec_entropy_gate_decode(logits[s_ % period], V, window, row_mask, 0.9, tau, tokens, decoded_out=decoded,
                                  max_entropy_out=maxh, decision_out=dec, workspace=ws_g, want_rows=False)
        ec.ec_select_recent_sliding(hist, state, masked, decoded, window, dec, k, idx)
        state_host.copy_(state, non_blocking=True)
        e3.record()
        torch.cuda.synchronize()                # the host reads skip_flag (and the row count): they shape the next step
        launches += 3
        st = state_host.numpy()
        skip = (st[:, 2] != 0) & (st[:, 3] <= n_cap)
        over_cap += int(((st[:, 2] != 0) & (st[:, 3] > n_cap)).sum())
        a, b_, c = e0.elapsed_time(e1) * 1e3, e1.elapsed_time(e2) * 1e3, e2.elapsed_time(e3) * 1e3
        if s_ > 0:
            t_skip += a; t_rec += b_; t_book += c
            n_skip += len(sk); n_rec += len(rc)
        per_step.append(dict(n_skip=len(sk), n_recompute=len(rc), rows=int(st[:, 3].max())))
        if int(masked.sum(dim=1).min().item()) < window:
            break
    us_skip = t_skip / max(n_skip * n_layers, 1)
    us_rec = t_rec / max(n_rec * n_layers, 1)
    steps_timed = max(len(per_step) - 1, 1)
    print(json.dumps({
        "trace": w.name, "mode": "sliding window, loop state on the device", "window": window, "k_recent": k,
        "n_cap": n_cap, "n_layers": n_layers, "n_steps": len(per_step), "batch": B, "tau": tau,
        "recompute_fraction": n_rec / max(n_skip + n_rec, 1),
        "us_per_layer_step_sequence": {"skip": us_skip, "recompute": us_rec},
        "skip_over_recompute": us_skip / us_rec if us_rec > 0 else None,
        "us_per_step_mean": {"attend_skip": t_skip / steps_timed, "attend_recompute": t_rec / steps_timed,
                             "gate_decode_and_select": t_book / steps_timed},
        "max_rows_of_a_partial_step": max(p_["rows"] for p_ in per_step), "steps_forced_full_by_capacity": over_cap,
        "gpu_launches": launches,
        "pattern": "".join("R" if p_["n_recompute"] == B else ("s" if p_["n_recompute"] == 0 else "m") for p_ in per_step),
        "timing": "CUDA events per step on the current stream, plain launches, host reads skip_flag every step"}))


def _run_only(args, torch, w, n_layers: int, dev) -> None:
    """Profiling aid: one part of the step over the same device workload (one CUDA graph
    per step, like the full run), a few iterations, one short JSON line."""
    wl = DeviceWorkload(w, n_layers, dev, seed=1234, need_recompute=args.only == "recompute")
    body = {"skip": lambda: [wl.attend_skip(l) for l in range(n_layers)],
            "recompute": lambda: [wl.attend_recompute(l) for l in range(n_layers)],
            "gate": lambda: [wl.gate(i) for i in range(wl.n_lbuf)]}[args.only]
    calls = wl.n_lbuf if args.only == "gate" else n_layers
    stream = torch.cuda.Stream(device=dev)
    ms = _graph_time(torch, body, max(args.steps, 1), max(args.warmup, 1), stream)
    print(json.dumps({"only": args.only, "workload": w.name, "calls_per_step": calls,
                      "us_per_call": ms * 1e3 / calls}))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(syn.WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="distinct K/V caches per step (0: enough to exceed 3x L2)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--trace", action="store_true",
                    help="full-depth step trace of the workload (its layers and steps; decisions from the gate)")
    ap.add_argument("--sliding", action="store_true",
                    help="with --trace: sliding-window decoding with the loop state on the device")
    ap.add_argument("--window", type=int, default=32, help="with --trace --sliding: window size (the paper: 8..128)")
    ap.add_argument("--trace-steps", type=int, default=0, help="with --trace: steps of the trace (0: the workload's)")
    ap.add_argument("--k-recent", type=int, default=-1,
                    help="recent-token budget k of the skip step (rows = block + k); default: the workload's own")
    ap.add_argument("--no-per-workload", action="store_true",
                    help="skip the per_workload section (the other benchmark shapes) of the JSON line")
    ap.add_argument("--only", default="", choices=["", "skip", "recompute", "gate"],
                    help="profiling aid: run only this part of the step")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
