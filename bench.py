#!/usr/bin/env python
"""Benchmark of the KVSink hot path on B200: sink prediction -> quantize/pack prefill -> one-token append ->
decode attention, through the C-ABI library, on seeded synthetic tensors shaped like the paper's workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Without --workload every workload runs in one process and rank 0 prints ONE JSON line: the headline numbers are those
of the largest single-GPU workload (the 32-layer decode step, 4 bit, with the 3-bit run beside it) and `per_workload`
holds the per-kernel times and roofline fractions of all of them.  With --workload NAME only that one runs and is the
headline.  With --impl reference the CPU oracle is timed instead, as it stands, on the host cores.

A "step" of a workload is one pass of the whole path:
  * 32-layer decode workload: predict_sinks once, quantize_append(T=S) into each of the 32 layer caches (the fp16
    prompt K/V of a layer is 8.6 GB, so one staging pair is reused for all layers), then 32 x (quantize_append(T=1)
    -> decode_attention), each on its own layer cache (69 / 87 GB of packed cache resident);
  * single-layer workloads: the same path over `--instances` layer-shaped instances (distinct inputs and caches, so
    that nothing a kernel reads is still in L2 from the previous kernel).
With --gpus N > 1 and no RANK in the environment the script starts N ranks itself (torch.distributed.run on 127.0.0.1).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2508_04257_b200 import synth  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
METRIC = "quantize+decode-attn achieved HBM GB/s"
HEADLINE = "decode32_4bit"
ALL_WORKLOADS = ("tiny", "llama2_7b_layer", "llama3_8b_gqa", "long_gqa", "decode32_3bit", "decode32_4bit")


# ------------------------------------------------------------------ algorithmic bytes
def quantize_bytes(wl, T):
    """fp16 K and V read once + packed codes + scale/zero written (bytes per layer)."""
    units = wl.batch * wl.n_kv_heads
    gv = min(wl.group, wl.head_dim)
    fp16_in = 2 * units * T * wl.head_dim * 2
    codes = 2 * units * T * wl.head_dim * wl.bits // 8
    k_params = 2 * 4 * units * (T // wl.group) * wl.head_dim
    v_params = 2 * 4 * units * T * (wl.head_dim // gv)
    return fp16_in + codes + k_params + v_params


def decode_bytes(wl, n):
    """Packed codes, scale/zero, sink mask and fp16 sink rows read once, q read, out written (per layer)."""
    units = wl.batch * wl.n_kv_heads
    gv = min(wl.group, wl.head_dim)
    per_token = 2 * wl.head_dim * wl.bits / 8 + 8 * wl.head_dim / wl.group + 8 * wl.head_dim / gv
    sinks = units * (wl.topk + wl.pfn_n) * wl.head_dim * 2 * 2
    qo = wl.batch * wl.n_q_heads * wl.head_dim * (2 + 4)
    return int(units * n * per_token + wl.batch * n / 8 + sinks + qo)


def predict_bytes(wl):
    """One 32-byte sector per token per listed channel, plus the 16-bit scores written and read."""
    return wl.batch * wl.seq * (len(wl.channels) * 32 + 4)


def append_bytes(wl):
    units = wl.batch * wl.n_kv_heads
    return units * wl.head_dim * (2 * 2 + 2 + 2 * wl.bits / 8) + units * 16


def step_bytes(wl, layers):
    return predict_bytes(wl) + layers * (quantize_bytes(wl, wl.seq) + append_bytes(wl) + decode_bytes(wl, wl.seq + 1))


def ncu_traffic(kernel_key, wl_name):
    """DRAM bytes per launch from the committed ncu capture of this kernel on this workload, or None when there is no
    capture or the kernel's source has changed since it was taken."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            rec = json.load(f)[f"{kernel_key}:{wl_name}"]
        for src, want in rec["sources_sha256"].items():
            with open(os.path.join(ROOT, "paper_2508_04257_b200", "csrc", src), "rb") as f:
                if hashlib.sha256(f.read()).hexdigest() != want:
                    return None
        return rec["dram_bytes_per_launch"]
    except Exception:
        return None


def workload_string(wl):
    s = (f"{wl.name}: B={wl.batch} Hq={wl.n_q_heads} Hkv={wl.n_kv_heads} D={wl.head_dim} S={wl.seq} bits={wl.bits} "
         f"G={wl.group} k={wl.topk} N={wl.pfn_n}")
    return s + (f" layers={wl.layers}" if wl.layers > 1 else "")


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) every millisecond while a timed region runs."""

    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x100: "display_clock_setting"}

    def __init__(self, device_index: int, period=0.001):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons, self.max_mhz = period, [], set(), None
        self._stop_evt, self._on = threading.Event(), threading.Event()
        self.h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    def run(self):
        while not self._stop_evt.is_set():
            if self.h is not None and self._on.is_set():
                try:
                    self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                    bits = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                    for b, name in self.REASONS.items():
                        if bits & b and name != "gpu_idle":
                            self.reasons.add(name)
                except Exception:
                    pass
            time.sleep(self.period)

    def region(self, on: bool):
        (self._on.set if on else self._on.clear)()

    def snapshot(self, reset=True):
        med = statistics.median(self.samples) if self.samples else None
        out = {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if reset:
            self.samples, self.reasons = [], set()
        return out

    def finish(self):
        self._stop_evt.set()


# ------------------------------------------------------------------ CPU oracle legs
def oracle_pass(wl, H, K, V, k1, v1, q, threads=None):
    """One pass of the path on the CPU oracle over host arrays; returns seconds per stage."""
    import oracle
    if threads:
        oracle.set_num_threads(threads)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk,
                        wl.pfn_n, wl.channels)
    t0 = time.perf_counter()
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    t1 = time.perf_counter()
    cache = oracle.Cache(cfg, bm, pos, cnt)
    t2 = time.perf_counter()
    oracle.quantize_append(cfg, cache, K, V)
    t3 = time.perf_counter()
    oracle.quantize_append(cfg, cache, k1, v1)
    t4 = time.perf_counter()
    oracle.decode_attention(cfg, cache, q)
    t5 = time.perf_counter()
    return {"predict": t1 - t0, "quantize": t3 - t2, "append": t4 - t3, "decode": t5 - t4, "threads": oracle.num_threads()}


def oracle_sample(wl, seqs, heads):
    """Host inputs for a bounded sample of the workload: one layer, the first `seqs` sequences x first `heads` KV heads."""
    rep = wl.n_q_heads // wl.n_kv_heads
    sub = wl.scaled(batch=min(seqs, wl.batch), n_kv_heads=heads, n_q_heads=heads * rep, layers=1)
    H = synth.make_hidden(sub).numpy()
    Kt, Vt = synth.make_kv(sub)
    k1, v1 = synth.make_new_token(sub)
    q = synth.make_query(sub, Kt).numpy()
    return sub, H, Kt.numpy(), Vt.numpy(), k1.numpy(), v1.numpy(), q


def sample_shape(wl, token_rows=1 << 20):
    """(sequences, KV heads) of a sample of about `token_rows` (sequence, KV head, token) rows: what the oracle gets
    through in about half a second per pass on sixteen cores."""
    heads = wl.n_kv_heads
    seqs = max(1, min(wl.batch, token_rows // (heads * wl.seq)))
    while seqs * heads * wl.seq > 2 * token_rows and heads > 1:
        heads //= 2
    return seqs, heads


def cpu_oracle_leg(wl, seconds, max_passes=64):
    """The oracle as it stands on the host cores, on a bounded one-layer sample, repeated for about `seconds`."""
    seqs, heads = sample_shape(wl)
    sub, H, K, V, k1, v1, q = oracle_sample(wl, seqs, heads)
    kinds = ("predict", "quantize", "append", "decode")
    st, n, t0 = None, 0, time.perf_counter()
    while n == 0 or (time.perf_counter() - t0 < seconds and n < max_passes):
        one = oracle_pass(sub, H, K, V, k1, v1, q)
        if st is None:
            st = one
        else:
            for k in kinds:
                st[k] += one[k]
        n += 1
    secs = sum(st[k] for k in kinds)
    sample = (f"{n} passes over one layer of {wl.name}, first {sub.batch} of {wl.batch} sequences x first {heads} of "
              f"{wl.n_kv_heads} KV heads (predict, prefill quantize, one append, one decode step each)")
    return {"value": n * step_bytes(sub, 1) / secs / 1e9, "unit": "GB/s", "cores": st["threads"], "kind": "oracle", "sample": sample,
            "seconds": secs, "stage_seconds": {k: st[k] for k in kinds}}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = synth.WORKLOADS[args.workload or HEADLINE]
    seqs, heads = sample_shape(wl, 1 << 18)
    sub, H, K, V, k1, v1, q = oracle_sample(wl, seqs, heads)
    for _ in range(min(args.warmup, 1)):
        oracle_pass(sub, H, K, V, k1, v1, q)
    steps = max(1, min(args.steps, 20))
    t0 = time.perf_counter()
    stages = None
    for _ in range(steps):
        stages = oracle_pass(sub, H, K, V, k1, v1, q)
    dt = (time.perf_counter() - t0) / steps
    gbs = step_bytes(sub, 1) / dt / 1e9
    sample = (f"per step one layer of {wl.name}, first {sub.batch} of {wl.batch} sequences x first {heads} of {wl.n_kv_heads} KV heads "
              "(predict, prefill quantize, one append, one decode step)")
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32 quantization / f64 attention", "data": "synthetic",
            "config": {"workload": workload_string(wl), "sample": sample},
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": stages["threads"], "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ the library's arm
class Bench:
    """One workload resident on the device: inputs, sink set, layer caches, and the step that runs the whole path."""

    def __init__(self, kv, wl, dev, instances):
        self.kv, self.wl, self.dev = kv, wl, dev
        self.layered = wl.layers > 1
        self.L = wl.layers if self.layered else instances
        self.n_in = 1 if self.layered else self.L           # distinct fp16 prompt inputs (one staging pair for 32 layers)
        L = self.L
        self.cfg = kv.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk,
                             wl.pfn_n, wl.channels)
        sz = kv.cache_sizes(self.cfg)
        self.H = synth.make_hidden(wl, dev)
        self.KV = [synth.make_kv(wl, l, dev) for l in range(self.n_in)]
        self.new = [synth.make_new_token(wl, l, 0, dev) for l in range(L)]
        self.qs = [synth.make_query(wl, self.KV[l % self.n_in][0], l) for l in range(L)]
        self.sinks = kv.SinkSet(self.cfg, dev)
        self.caches = [kv.KVCache(self.cfg, self.sinks, dev) for _ in range(L)]
        self.outs = [torch.empty((wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device=dev) for _ in range(L)]
        self.ws_p = torch.empty(sz["predict_workspace_bytes"], dtype=torch.uint8, device=dev)
        self.ws_d = torch.empty(sz["decode_workspace_bytes"], dtype=torch.uint8, device=dev)
        self.kinds = ("predict", "quantize", "append", "decode")
        self.ev = {k: [] for k in self.kinds}      # (start event, end event, calls between them)

    def _timed(self, kind, fn, calls, record):
        if record:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            self.ev[kind].append((a, b, calls))
        else:
            fn()

    def step(self, record):
        kv, cfg, L = self.kv, self.cfg, self.L
        self._timed("predict", lambda: kv.predict_sinks(cfg, self.H, self.sinks, self.ws_p), 1, record)

        def quantize_all():
            for l in range(L):
                self.caches[l].seq_len = 0
                K, V = self.KV[l % self.n_in]
                kv.quantize_append(cfg, self.caches[l], K, V)

        append = lambda l: kv.quantize_append(cfg, self.caches[l], self.new[l][0], self.new[l][1])
        decode = lambda l: kv.decode_attention(cfg, self.caches[l], self.qs[l], self.outs[l], None, self.ws_d, want_lse=False)
        self._timed("quantize", quantize_all, L, record)
        if self.layered:
            # the decode step of the model: layer by layer, the new token appended, then attended
            for l in range(L):
                self._timed("append", lambda: append(l), 1, record)
                self._timed("decode", lambda: decode(l), 1, record)
        else:
            # independent instances: the appends, then the decode launches back to back (one event pair around each run,
            # so that an event between two launches does not undo their programmatic overlap)
            self._timed("append", lambda: [append(l) for l in range(L)], L, record)
            self._timed("decode", lambda: [decode(l) for l in range(L)], L, record)

    def kind_us(self):
        """Average microseconds per call of each kind over the recorded steps."""
        out = {}
        for k in self.kinds:
            ms = sum(a.elapsed_time(b) for a, b, _ in self.ev[k])
            n = sum(c for _, _, c in self.ev[k])
            out[k] = ms * 1e3 / max(n, 1)
        return out

    def run(self, steps, warmup, barrier, sampler, max_over_ranks):
        for _ in range(warmup):
            self.step(False)
        barrier()
        n0 = self.kv.launch_count()
        if sampler is not None:
            sampler.region(True)
        t_a, t_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_a.record()
        for _ in range(steps):
            self.step(True)
        t_b.record()
        barrier()
        if sampler is not None:
            sampler.region(False)
        launches = self.kv.launch_count() - n0
        ms_step = max_over_ranks(t_a.elapsed_time(t_b)) / steps
        return ms_step, launches

    def e2e(self, steps, barrier, max_over_ranks):
        """The same step through the same calls, its inputs copied from pinned host memory and its results copied back."""
        wl, L = self.wl, self.L
        pin = lambda t: t.cpu().pin_memory()
        hH = pin(self.H)
        hKV = [(pin(a), pin(b)) for a, b in self.KV]
        hnew = [(pin(a), pin(b)) for a, b in self.new]
        hq = [pin(x) for x in self.qs]
        host_out = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in self.outs]
        kv, cfg = self.kv, self.cfg
        h2d = hH.numel() * 2 + L * sum(a.numel() * 2 + b.numel() * 2 for a, b in hKV) // self.n_in
        h2d += sum(a.numel() * 4 for a, _ in hnew) + sum(x.numel() * 2 for x in hq)
        d2h = sum(o.numel() * 4 for o in self.outs)

        def one():
            self.H.copy_(hH, non_blocking=True)
            kv.predict_sinks(cfg, self.H, self.sinks, self.ws_p)
            for l in range(L):          # a layer's prompt K/V arrives from the host, then is quantized into its cache
                K, V = self.KV[l % self.n_in]
                K.copy_(hKV[l % self.n_in][0], non_blocking=True)
                V.copy_(hKV[l % self.n_in][1], non_blocking=True)
                self.caches[l].seq_len = 0
                kv.quantize_append(cfg, self.caches[l], K, V)
            for l in range(L):
                self.new[l][0].copy_(hnew[l][0], non_blocking=True)
                self.new[l][1].copy_(hnew[l][1], non_blocking=True)
                self.qs[l].copy_(hq[l], non_blocking=True)
                kv.quantize_append(cfg, self.caches[l], self.new[l][0], self.new[l][1])
                kv.decode_attention(cfg, self.caches[l], self.qs[l], self.outs[l], None, self.ws_d, want_lse=False)
                host_out[l].copy_(self.outs[l], non_blocking=True)

        one()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            one()
        b.record()
        barrier()
        ms = max_over_ranks(a.elapsed_time(b)) / steps
        return ms, int(h2d), int(d2h)


def calibrated_record(kv, wl, dev, instances, steps, warmup, peak):
    """The static-parameter variant of a single-layer workload: calibration on the prompt itself, then per instance
    quantize_append_calibrated(T=S), one appended token and decode_attention_calibrated (kernel times only)."""
    cfg = kv.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n, wl.channels)
    L = instances
    H = synth.make_hidden(wl, dev)
    KV = [synth.make_kv(wl, l, dev) for l in range(L)]
    new = [synth.make_new_token(wl, l, 0, dev) for l in range(L)]
    qs = [synth.make_query(wl, KV[l][0], l) for l in range(L)]
    sinks = kv.SinkSet(cfg, dev)
    kv.predict_sinks(cfg, H, sinks)
    caches = [kv.KVCache(cfg, sinks, dev) for _ in range(L)]
    params = kv.StaticParams(cfg, dev)
    outs = [torch.empty((wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device=dev) for _ in range(L)]
    ws_d = torch.empty(kv.cache_sizes(cfg)["decode_workspace_bytes"], dtype=torch.uint8, device=dev)
    ev = {"calibrate": [], "quantize": [], "decode": []}

    def timed(kind, fn, rec):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        if rec:
            ev[kind].append((a, b))

    def quantize_all():
        for l in range(L):
            caches[l].seq_len = 0
            kv.quantize_append_calibrated(cfg, caches[l], params, KV[l][0], KV[l][1])

    def decode_all():
        for l in range(L):
            kv.decode_attention_calibrated(cfg, caches[l], params, qs[l], outs[l], None, ws_d, want_lse=False)

    for it in range(warmup + steps):
        rec = it >= warmup
        timed("calibrate", lambda: kv.calibrate(cfg, KV[0][0], KV[0][1], sinks, params), rec)
        timed("quantize", quantize_all, rec)
        for l in range(L):
            kv.quantize_append_calibrated(cfg, caches[l], params, new[l][0], new[l][1])
        timed("decode", decode_all, rec)
    torch.cuda.synchronize()
    us = {k: sum(a.elapsed_time(b) for a, b in v) * 1e3 / len(v) / (1 if k == "calibrate" else L) for k, v in ev.items()}
    units, n = wl.batch * wl.n_kv_heads, wl.seq + 1
    code_bytes = 2 * units * wl.head_dim * wl.bits // 8
    qb = 2 * units * wl.seq * wl.head_dim * 2 + code_bytes * wl.seq
    db = code_bytes * n + wl.batch * n // 8 + units * (wl.topk + wl.pfn_n) * wl.head_dim * 4 + wl.batch * wl.n_q_heads * wl.head_dim * 6
    cb = 2 * units * wl.seq * wl.head_dim * 2
    gbs = lambda bytes_, t: bytes_ / (t * 1e-6) / 1e9
    return {"workload": workload_string(wl) + " (static parameters)", "instances_per_step": L, "calibrate_us": us["calibrate"],
            "quantize_us": us["quantize"], "decode_us": us["decode"], "device_status": kv.read_status(caches[0]),
            "calibrate": {"algorithmic_bytes": cb, "GBs": gbs(cb, us["calibrate"]), "frac_of_measured_peak": gbs(cb, us["calibrate"]) / peak},
            "quantize": {"algorithmic_bytes": qb, "GBs": gbs(qb, us["quantize"]), "frac_of_measured_peak": gbs(qb, us["quantize"]) / peak},
            "decode": {"algorithmic_bytes": db, "GBs": gbs(db, us["decode"]), "frac_of_measured_peak": gbs(db, us["decode"]) / peak}}


def pertoken_record(kv, wl, dev, instances, steps, warmup, peak):
    """The per-token key variant of a single-layer workload: per instance quantize_append_pertoken(T=S), one appended
    token and decode_attention_pertoken (kernel times only)."""
    cfg = kv.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n, wl.channels)
    L = instances
    H = synth.make_hidden(wl, dev)
    KV = [synth.make_kv(wl, l, dev) for l in range(L)]
    new = [synth.make_new_token(wl, l, 0, dev) for l in range(L)]
    qs = [synth.make_query(wl, KV[l][0], l) for l in range(L)]
    sinks = kv.SinkSet(cfg, dev)
    kv.predict_sinks(cfg, H, sinks)
    caches = [kv.KVCache(cfg, sinks, dev, per_token_keys=True) for _ in range(L)]
    outs = [torch.empty((wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device=dev) for _ in range(L)]
    ws_d = torch.empty(kv.cache_sizes(cfg)["decode_workspace_bytes"], dtype=torch.uint8, device=dev)
    ev = {"quantize": [], "decode": []}

    def timed(kind, fn, rec):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        if rec:
            ev[kind].append((a, b))

    def quantize_all():
        for l in range(L):
            caches[l].seq_len = 0
            kv.quantize_append_pertoken(cfg, caches[l], KV[l][0], KV[l][1])

    def decode_all():
        for l in range(L):
            kv.decode_attention_pertoken(cfg, caches[l], qs[l], outs[l], None, ws_d, want_lse=False)

    for it in range(warmup + steps):
        rec = it >= warmup
        timed("quantize", quantize_all, rec)
        for l in range(L):
            kv.quantize_append_pertoken(cfg, caches[l], new[l][0], new[l][1])
        timed("decode", decode_all, rec)
    torch.cuda.synchronize()
    us = {k: sum(a.elapsed_time(b) for a, b in v) * 1e3 / len(v) / L for k, v in ev.items()}
    units, n = wl.batch * wl.n_kv_heads, wl.seq + 1
    ngv = wl.head_dim // min(wl.group, wl.head_dim)
    tok_bytes = 2 * wl.head_dim * wl.bits // 8 + 4 * 4 * ngv          # codes of K and V, (scale, zero) of both per channel group
    qb = units * wl.seq * (2 * wl.head_dim * 2 + tok_bytes)
    db = units * n * tok_bytes + wl.batch * n // 8 + units * (wl.topk + wl.pfn_n) * wl.head_dim * 4 + wl.batch * wl.n_q_heads * wl.head_dim * 6
    gbs = lambda bytes_, t: bytes_ / (t * 1e-6) / 1e9
    return {"workload": workload_string(wl) + " (per-token keys)", "instances_per_step": L, "quantize_us": us["quantize"],
            "decode_us": us["decode"], "device_status": kv.read_status(caches[0]),
            "quantize": {"algorithmic_bytes": qb, "GBs": gbs(qb, us["quantize"]), "frac_of_measured_peak": gbs(qb, us["quantize"]) / peak},
            "decode": {"algorithmic_bytes": db, "GBs": gbs(db, us["decode"]), "frac_of_measured_peak": gbs(db, us["decode"]) / peak}}


def prefill_attention_record(kv, wl, dev, steps, warmup):
    """Attention of every prompt query over the just-quantized cache of a single-layer workload (kernel time only)."""
    cfg = kv.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n, wl.channels)
    H = synth.make_hidden(wl, dev)
    K, V = synth.make_kv(wl, 0, dev)
    sinks = kv.SinkSet(cfg, dev)
    kv.predict_sinks(cfg, H, sinks)
    cache = kv.KVCache(cfg, sinks, dev)
    kv.quantize_append(cfg, cache, K, V)
    del H
    g = torch.Generator(device=dev)
    g.manual_seed(wl.seed + 77)
    q = torch.randn((wl.batch, wl.n_q_heads, wl.seq, wl.head_dim), device=dev, generator=g).half()
    out = torch.empty((wl.batch, wl.n_q_heads, wl.seq, wl.head_dim), dtype=torch.float32, device=dev)
    for _ in range(warmup):
        kv.prefill_attention(cfg, cache, q, 0, out, None, want_lse=False)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        kv.prefill_attention(cfg, cache, q, 0, out, None, want_lse=False)
    b.record()
    torch.cuda.synchronize()
    us = a.elapsed_time(b) * 1e3 / steps
    flop = 4.0 * wl.batch * wl.n_q_heads * wl.head_dim * wl.seq * (wl.seq + 1) / 2        # QK^T and PV over the causal triangle
    return {"workload": workload_string(wl) + " (attention of all prompt queries over the quantized cache)", "prefill_attention_us": us,
            "attention_tflops": flop / (us * 1e-6) / 1e12, "device_status": kv.read_status(cache)}


def workload_record(b: Bench, ms_step, launches, steps, peak, world, agg):
    wl = b.wl
    us = b.kind_us()
    qb, db = quantize_bytes(wl, wl.seq), decode_bytes(wl, wl.seq + 1)
    q_gbs, d_gbs = qb / (us["quantize"] * 1e-6) / 1e9, db / (us["decode"] * 1e-6) / 1e9
    rec = {"workload": workload_string(wl), "layers_or_instances_per_step": b.L, "ms_per_step": ms_step,
           "value_GBs": agg(step_bytes(wl, b.L), world, ms_step * 1e-3) / 1e9, "gpu_launches_per_step": launches / steps,
           "quantize_us": us["quantize"], "decode_us": us["decode"], "append_us": us["append"], "predict_us": us["predict"],
           "quantize": {"algorithmic_bytes": qb, "GBs": q_gbs, "frac_of_measured_peak": q_gbs / peak, "pct_of_8TBs": 100 * q_gbs / NOMINAL_HBM_GBS},
           "decode": {"algorithmic_bytes": db, "GBs": d_gbs, "frac_of_measured_peak": d_gbs / peak, "pct_of_8TBs": 100 * d_gbs / NOMINAL_HBM_GBS}}
    if b.layered:
        rec["decode_us_per_step"] = b.L * (us["append"] + us["decode"])     # all layers: append + attend
    return rec, us, q_gbs, d_gbs, qb, db


def spawn_ranks(args):
    """--gpus N > 1 without a launcher: start N ranks of this script under torch.distributed.run on 127.0.0.1."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_plumbing_only(args):
    """The multi-rank plumbing alone, on CPU over gloo (no kernels, no timing claim): rendezvous, barrier, max over ranks and
    the aggregate; rank 0 prints the line's rank-dependent fields.  What the multi-process CPU test drives."""
    import torch.distributed as dist
    from paper_2508_04257_b200 import dist_util
    ri = dist_util.rank_info()
    if ri.world > 1:
        dist.init_process_group("gloo")
    wl = synth.WORKLOADS["tiny"].scaled(seed=dist_util.rank_seed(synth.WORKLOADS["tiny"].seed, ri.rank))
    if ri.world > 1:
        dist.barrier()
    ms = dist_util.max_over_ranks(1.0 + ri.rank, "cpu")
    value = dist_util.aggregate_throughput(step_bytes(wl, 1), ri.world, ms * 1e-3) / 1e9
    if ri.rank == 0:
        print(json.dumps({"plumbing_only": True, "metric": METRIC, "n_gpus": ri.world, "ms_per_step": ms, "value": value, "unit": "GB/s",
                          "scaling": "weak"}), flush=True)
    if ri.world > 1:
        dist.destroy_process_group()


def run_ours(args):
    import torch.distributed as dist
    import paper_2508_04257_b200 as kv
    from paper_2508_04257_b200 import dist_util

    ri = dist_util.rank_info()
    rank, world, local = ri.rank, ri.world, ri.local_rank
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    max_over = lambda ms: dist_util.max_over_ranks(ms, dev)
    peak, peak_kind = measured_peak()
    names = [args.workload] if args.workload else list(ALL_WORKLOADS)
    headline = args.workload or HEADLINE
    warmup = max(args.warmup, 3)
    sampler = ClockSampler(local)
    sampler.start()
    per, head = {}, None
    for name in names:
        base = synth.WORKLOADS[name]
        wl = base.scaled(seed=dist_util.rank_seed(base.seed, rank))
        if args.batch > 0:
            wl = wl.scaled(batch=args.batch)
        if args.layers > 0 and wl.layers > 1:
            wl = wl.scaled(layers=args.layers)
        b = Bench(kv, wl, dev, args.instances)
        is_head = name == headline
        # the headline workload runs --steps steps; the others a number of steps that lasts a comparable, short time
        steps = args.steps if is_head else max(args.steps, 20 if wl.layers == 1 else 3)
        ms_step, launches = b.run(steps, warmup, barrier, sampler if is_head else None, max_over)
        rec, us, q_gbs, d_gbs, qb, db = workload_record(b, ms_step, launches, steps, peak, world, dist_util.aggregate_throughput)
        rec["device_status"] = kv.read_status(b.caches[0])
        if is_head:
            e2e = None
            if args.e2e_steps > 0:
                ms, h2d, d2h = b.e2e(args.e2e_steps, barrier, max_over)
                e2e = {"value": dist_util.aggregate_throughput(step_bytes(wl, b.L), world, ms * 1e-3) / 1e9, "unit": "GB/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms, "steps": args.e2e_steps}
            head = dict(wl=wl, rec=rec, us=us, q_gbs=q_gbs, d_gbs=d_gbs, qb=qb, db=db, ms_step=ms_step, launches=launches, steps=steps,
                        L=b.L, e2e=e2e, clocks=sampler.snapshot(), layered=b.layered)
        per[name] = rec
        del b
        torch.cuda.empty_cache()
    if not args.workload:
        # the next scope rows on the LLaMA2-7B-shaped layer: static (calibrated) parameters, per-token keys, prompt attention
        base = synth.WORKLOADS["llama2_7b_layer"]
        per["llama2_7b_layer_static"] = calibrated_record(kv, base.scaled(seed=dist_util.rank_seed(base.seed, rank)), dev, args.instances, 20, warmup, peak)
        torch.cuda.empty_cache()
        per["llama2_7b_layer_pertoken_keys"] = pertoken_record(kv, base.scaled(seed=dist_util.rank_seed(base.seed, rank)), dev, args.instances, 20, warmup, peak)
        torch.cuda.empty_cache()
        per["llama2_7b_layer_prefill_attention"] = prefill_attention_record(kv, base.scaled(seed=dist_util.rank_seed(base.seed, rank)), dev, 3, 1)
        torch.cuda.empty_cache()
    sampler.finish()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    wl = head["wl"]
    roof = {"bound": "hbm", "kernel": "quantize_bulk_kernel (prefill quantize + pack + sink compaction)", "achieved": head["q_gbs"], "peak": peak,
            "peak_kind": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": head["q_gbs"] / peak,
            "frac_of_nominal_8TBs": head["q_gbs"] / NOMINAL_HBM_GBS, "algorithmic_bytes_per_launch": head["qb"],
            "us_per_launch": head["us"]["quantize"], "traffic": ncu_traffic("quantize_bulk_kernel", wl.name) if args.batch == 0 else None}
    roof_d = {"bound": "hbm", "kernel": "decode_kernel (+ decode_merge_kernel beyond eight splits)", "achieved": head["d_gbs"], "peak": peak,
              "unit": "GB/s", "frac": head["d_gbs"] / peak, "frac_of_nominal_8TBs": head["d_gbs"] / NOMINAL_HBM_GBS,
              "algorithmic_bytes_per_launch": head["db"], "us_per_launch": head["us"]["decode"],
              "traffic": ncu_traffic("decode_kernel", wl.name) if args.batch == 0 else None}
    cpu = cpu_oracle_leg(synth.WORKLOADS[headline], args.cpu_seconds) if (world == 1 and args.cpu_seconds > 0) else None
    if head["layered"]:
        step_text = (f"predict_sinks once; quantize_append(T=S) into each of the {head['L']} layer caches from one reused fp16 staging pair; "
                     f"then {head['L']} x (quantize_append(T=1) -> decode_attention), every layer on its own resident cache")
        l2 = f"{head['L']} layer caches resident, {step_bytes(wl, head['L']) / 1e9:.1f} GB touched per step: every kernel's input is far larger than L2"
    else:
        step_text = "predict_sinks, then per instance quantize_append(T=S), then per instance quantize_append(T=1), then per instance decode_attention"
        l2 = (f"inputs larger than L2: {head['L']} instances, {step_bytes(wl, head['L']) / 1e6:.0f} MB touched per step; each kernel reads data "
              "last touched more than 300 MB of traffic earlier")
    line = {"metric": METRIC, "value": head["rec"]["value_GBs"], "unit": "GB/s", "n_gpus": world, "steps": head["steps"],
            "warmup": warmup, "ms_per_step": head["ms_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_string(wl), "layers_or_instances_per_step": head["L"], "l2": l2, "step": step_text},
            "decode_us_per_step": head["rec"].get("decode_us_per_step", head["us"]["decode"]),
            "decode_us_per_layer": head["us"]["decode"], "append_us": head["us"]["append"], "predict_us": head["us"]["predict"],
            "quantize_us": head["us"]["quantize"],
            "pct_of_8TBs": {"quantize": 100 * head["q_gbs"] / NOMINAL_HBM_GBS, "decode": 100 * head["d_gbs"] / NOMINAL_HBM_GBS},
            "roofline": roof, "roofline_decode": roof_d, "cpu_baseline": cpu, "e2e": head["e2e"], "gpu_launches": int(head["launches"]),
            "clocks": head["clocks"], "device_status": head["rec"]["device_status"], "per_workload": per}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=12, help="timed steps of the headline workload")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(synth.WORKLOADS), help="run only this workload (default: all)")
    ap.add_argument("--instances", type=int, default=4, help="layer-shaped instances per step of a single-layer workload")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count of the 32-layer workload (profiling a smaller case)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling a smaller case)")
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU work to time for the oracle baseline (0 = skip)")
    ap.add_argument("--plumbing-only", action="store_true", help="multi-rank plumbing on CPU over gloo, no kernels")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(spawn_ranks(args))
    if args.plumbing_only:
        run_plumbing_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
