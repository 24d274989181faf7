#!/usr/bin/env python
"""Benchmark of the KVSink hot path on B200: sink prediction -> quantize/pack prefill -> one-token append ->
decode attention, through the C-ABI library, on seeded synthetic tensors shaped like the paper's workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

One "step" is one pass of the whole path over `--instances` layer-shaped instances of the workload (distinct
inputs and caches, so that nothing a kernel reads is still in L2 from the previous kernel).  Rank 0 prints ONE
JSON line.  With --impl reference the CPU oracle is timed instead, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
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


# ------------------------------------------------------------------ algorithmic bytes
def quantize_bytes(wl, T):
    """fp16 K and V read once + packed codes + scale/zero written (bytes per layer instance)."""
    units = wl.batch * wl.n_kv_heads
    gv = min(wl.group, wl.head_dim)
    fp16_in = 2 * units * T * wl.head_dim * 2
    codes = 2 * units * T * wl.head_dim * wl.bits // 8
    k_params = 2 * 4 * units * (T // wl.group) * wl.head_dim
    v_params = 2 * 4 * units * T * (wl.head_dim // gv)
    return fp16_in + codes + k_params + v_params


def decode_bytes(wl, n):
    """Packed codes, scale/zero, sink mask and fp16 sink rows read once, q read, out written (per layer instance)."""
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


def step_bytes(wl, instances):
    return predict_bytes(wl) + instances * (quantize_bytes(wl, wl.seq) + append_bytes(wl) + decode_bytes(wl, wl.seq + 1))


def ncu_traffic(kernel_key):
    """DRAM bytes per launch from the committed ncu capture, or None once the kernel's source has changed since."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            rec = json.load(f)[kernel_key]
        src = os.path.join(ROOT, "paper_2508_04257_b200", "csrc", rec["source"])
        with open(src, "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != rec["source_sha256"]:
                return None
        return rec["dram_bytes_per_launch"]
    except Exception:
        return None


def workload_string(wl):
    return (f"{wl.name}: B={wl.batch} Hq={wl.n_q_heads} Hkv={wl.n_kv_heads} D={wl.head_dim} S={wl.seq} bits={wl.bits} "
            f"G={wl.group} k={wl.topk} N={wl.pfn_n}")


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x100: "display_clock_setting"}

    def __init__(self, device_index: int, period=0.02):
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

    def finish(self):
        self._stop_evt.set()
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


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


def oracle_sample(wl, heads):
    """Host inputs for a bounded sample of the workload: every sequence, the first `heads` KV heads."""
    rep = wl.n_q_heads // wl.n_kv_heads
    sub = wl.scaled(n_kv_heads=heads, n_q_heads=heads * rep)
    H = synth.make_hidden(sub).numpy()
    Kt, Vt = synth.make_kv(sub)
    k1, v1 = synth.make_new_token(sub)
    q = synth.make_query(sub, Kt).numpy()
    return sub, H, Kt.numpy(), Vt.numpy(), k1.numpy(), v1.numpy(), q


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = synth.WORKLOADS[args.workload]
    heads = min(wl.n_kv_heads, args.ref_heads)
    sub, H, K, V, k1, v1, q = oracle_sample(wl, heads)
    for _ in range(min(args.warmup, 1)):
        oracle_pass(sub, H, K, V, k1, v1, q)
    t0 = time.perf_counter()
    stages = None
    for _ in range(args.steps):
        stages = oracle_pass(sub, H, K, V, k1, v1, q)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    gbs = step_bytes(sub, 1) / dt / 1e9
    sample = f"1 instance, all {wl.batch} sequences x first {heads} of {wl.n_kv_heads} KV heads of {wl.name} per step"
    line = {"impl": "reference", "metric": "quantize+decode-attn achieved HBM GB/s", "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32 quantization / f64 attention", "data": "synthetic",
            "config": {"workload": workload_string(wl), "sample": sample},
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": stages["threads"], "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ the library's arm
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

    wl = synth.WORKLOADS[args.workload].scaled(seed=dist_util.rank_seed(synth.WORKLOADS[args.workload].seed, rank))
    if args.batch > 0:
        wl = wl.scaled(batch=args.batch)
    L = args.instances
    cfg = kv.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                    wl.channels)
    sz = kv.cache_sizes(cfg)
    H = synth.make_hidden(wl, dev)
    KV = [synth.make_kv(wl, l, dev) for l in range(L)]
    new = [synth.make_new_token(wl, l, 0, dev) for l in range(L)]
    qs = [synth.make_query(wl, KV[l][0], l) for l in range(L)]
    sinks = kv.SinkSet(cfg, dev)
    caches = [kv.KVCache(cfg, sinks, dev) for _ in range(L)]
    outs = [torch.empty((wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device=dev) for _ in range(L)]
    ws_p = torch.empty(sz["predict_workspace_bytes"], dtype=torch.uint8, device=dev)
    ws_d = torch.empty(sz["decode_workspace_bytes"], dtype=torch.uint8, device=dev)

    kinds = ("predict", "quantize", "append", "decode")
    ev = {k: [] for k in kinds}

    def timed(kind, fn, record):
        if record:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            ev[kind].append((a, b))
        else:
            fn()

    def step(record, H_=H, KV_=KV, new_=new, qs_=qs):
        timed("predict", lambda: kv.predict_sinks(cfg, H_, sinks, ws_p), record)
        for l in range(L):
            caches[l].seq_len = 0
            timed("quantize", lambda: kv.quantize_append(cfg, caches[l], KV_[l][0], KV_[l][1]), record)
        for l in range(L):
            timed("append", lambda: kv.quantize_append(cfg, caches[l], new_[l][0], new_[l][1]), record)
            timed("decode", lambda: kv.decode_attention(cfg, caches[l], qs_[l], outs[l], None, ws_d, want_lse=False), record)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step(False)
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    sampler.region(True)
    t_a, t_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_a.record()
    for _ in range(args.steps):
        step(True)
    t_b.record()
    barrier()
    sampler.region(False)
    clocks = sampler.finish()
    ms_total = dist_util.max_over_ranks(t_a.elapsed_time(t_b), dev)
    ms_step = ms_total / args.steps
    kind_ms = {k: sum(a.elapsed_time(b) for a, b in ev[k]) / max(len(ev[k]), 1) for k in kinds}   # per call
    bytes_step = step_bytes(wl, L)
    value = dist_util.aggregate_throughput(bytes_step, world, ms_step * 1e-3) / 1e9
    status = kv.read_status(caches[0])

    # ---- end to end: pinned host inputs copied in, result copied out, every step
    e2e = None
    if args.e2e_steps > 0:
        pin = lambda t: t.cpu().pin_memory()
        hH, hKV, hnew, hq = pin(H), [(pin(a), pin(b)) for a, b in KV], [(pin(a), pin(b)) for a, b in new], [pin(x) for x in qs]
        host_out = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in outs]
        h2d = hH.numel() * 2 + sum(a.numel() * 2 + b.numel() * 2 for a, b in hKV) + sum(a.numel() * 4 for a, _ in hnew) + sum(x.numel() * 2 for x in hq)
        d2h = sum(o.numel() * 4 for o in outs)

        def e2e_step():
            H.copy_(hH, non_blocking=True)
            for l in range(L):
                KV[l][0].copy_(hKV[l][0], non_blocking=True)
                KV[l][1].copy_(hKV[l][1], non_blocking=True)
                new[l][0].copy_(hnew[l][0], non_blocking=True)
                new[l][1].copy_(hnew[l][1], non_blocking=True)
                qs[l].copy_(hq[l], non_blocking=True)
            step(False)
            for l in range(L):
                host_out[l].copy_(outs[l], non_blocking=True)

        e2e_step()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        b.record()
        barrier()
        ms = dist_util.max_over_ranks(a.elapsed_time(b), dev)
        e2e = {"value": dist_util.aggregate_throughput(bytes_step, world, ms / args.e2e_steps * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": ms / args.e2e_steps, "steps": args.e2e_steps}
        del hH, hKV, hnew, hq

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    qb, db = quantize_bytes(wl, wl.seq), decode_bytes(wl, wl.seq + 1)
    q_gbs, d_gbs = qb / (kind_ms["quantize"] * 1e-3) / 1e9, db / (kind_ms["decode"] * 1e-3) / 1e9
    roof = {"bound": "hbm", "kernel": "quantize_bulk_kernel (prefill quantize + pack + sink compaction)", "achieved": q_gbs, "peak": peak,
            "peak_kind": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": q_gbs / peak, "frac_of_nominal_8TBs": q_gbs / NOMINAL_HBM_GBS,
            "algorithmic_bytes_per_launch": qb, "us_per_launch": kind_ms["quantize"] * 1e3,
            "traffic": ncu_traffic("quantize_bulk_kernel") if args.workload == "llama2_7b_layer" and args.batch == 0 else None}
    roof_d = {"bound": "hbm", "kernel": "decode_kernel (+ decode_merge_kernel beyond eight splits)", "achieved": d_gbs, "peak": peak, "unit": "GB/s",
              "frac": d_gbs / peak, "frac_of_nominal_8TBs": d_gbs / NOMINAL_HBM_GBS, "algorithmic_bytes_per_launch": db,
              "us_per_launch": kind_ms["decode"] * 1e3,
              "traffic": ncu_traffic("decode_kernel") if args.workload == "llama2_7b_layer" and args.batch == 0 else None}

    cpu = None
    if world == 1 and args.cpu_heads > 0:
        # the oracle as it stands on the host cores: whole steps (predict once, then every instance) over the sample,
        # repeated until about ten seconds of CPU work have been timed
        heads = min(wl.n_kv_heads, args.cpu_heads)
        sub, hH2, hK, hV, hk1, hv1, hq2 = oracle_sample(synth.WORKLOADS[args.workload], heads)
        st, steps_done, t_cpu0 = None, 0, time.perf_counter()
        while steps_done == 0 or (time.perf_counter() - t_cpu0 < args.cpu_seconds and steps_done < 64):
            one = oracle_pass(sub, hH2, hK, hV, hk1, hv1, hq2)
            for _ in range(L - 1):          # the step has L instances: time the oracle on as many passes
                more = oracle_pass(sub, hH2, hK, hV, hk1, hv1, hq2)
                for k in ("quantize", "append", "decode"):
                    one[k] += more[k]
            if st is None:
                st = one
            else:
                for k in kinds:
                    st[k] += one[k]
            steps_done += 1
        secs = st["predict"] + st["quantize"] + st["append"] + st["decode"]
        cpu = {"value": steps_done * step_bytes(sub, L) / secs / 1e9, "unit": "GB/s", "cores": st["threads"], "kind": "oracle",
               "sample": f"{steps_done} steps of {L} instances, all {wl.batch} sequences x first {heads} of {wl.n_kv_heads} KV heads of {wl.name}",
               "seconds": secs, "stage_seconds": {k: st[k] for k in kinds}}

    # predict: score + select; per instance: bulk quantize, append, decode.  Decode is one kernel when a unit has at most
    # eight sequence splits (they merge inside a thread-block cluster: configs 2 and 4), else split kernel + merge kernel.
    decode_launches = 1 if args.workload in ("llama2_7b_layer", "decode32_3bit", "decode32_4bit", "tiny") else 2
    launches_per_step = 2 + L * (1 + 1 + decode_launches)
    line = {"metric": "quantize+decode-attn achieved HBM GB/s", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_string(wl), "instances_per_step": L,
                       "l2": f"inputs larger than L2: {L} instances, {bytes_step / 1e6:.0f} MB touched per step; each kernel reads data "
                             "last touched more than 300 MB of traffic earlier",
                       "step": "predict_sinks, then per instance quantize_append(T=S), then per instance quantize_append(T=1) + decode_attention"},
            "decode_us_per_step": kind_ms["decode"] * 1e3, "append_us": kind_ms["append"] * 1e3, "predict_us": kind_ms["predict"] * 1e3,
            "quantize_us": kind_ms["quantize"] * 1e3, "pct_of_8TBs": {"quantize": 100 * q_gbs / NOMINAL_HBM_GBS, "decode": 100 * d_gbs / NOMINAL_HBM_GBS},
            "roofline": roof, "roofline_decode": roof_d, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks, "device_status": status}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b_layer", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--instances", type=int, default=4, help="layer-shaped instances per step")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling a smaller case)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-heads", type=int, default=32, help="KV heads in the CPU-oracle sample (0 = skip)")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU work to time for the oracle baseline")
    ap.add_argument("--ref-heads", type=int, default=4, help="KV heads per step of --impl reference")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
