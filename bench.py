#!/usr/bin/env python
"""Benchmark of libqknorm's hot path: layerwise QK-RMSNorm through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload C5] [--no-table]

One "step" is one pass of the whole hot path (load, per-shard sum of squares,
combine, gamma multiply, scale, store; Q and K in one launch) over one batch of
synthetic input of the named workload.  Rank 0 prints ONE JSON line.

 * value        whole-job GB/s (algorithmic bytes: every element read once and
                written once, every gamma read once), inputs resident in HBM.
 * e2e          the same metric when every step also copies that step's inputs
                from pinned host memory and reads the result back.
 * roofline     the kernel against the measured HBM copy rate of this machine.
 * cpu_baseline the fp64 CPU oracle, timed on this machine's host cores on a bounded
                sample of the same workload (a reported baseline, not a target).
 * configs      the other workloads (us/call, GB/s, fraction of the HBM peak;
                decode sizes also under CUDA-graph replay).

With N > 1 (torchrun) every rank runs the same workload on its own GPU on its
own tokens: the path shards by token range with no exchange, so there is no
collective on the data path ("scaling": "weak").

--impl reference times the CPU oracle as it stands (there is no other
implementation of the paper to run): rank 0 only, each step a bounded sample.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2608_09160_b200 import workloads as W  # noqa: E402

METRIC = "qknorm_prefill_GBps"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126e6          # B200 L2 capacity
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes (read + write) per launch of the dominant kernel, measured by ncu
# (dram__bytes_read.sum + dram__bytes_write.sum).  The figures live in the profile summaries under
# profiles/ (a line "traffic_bytes_per_launch = N"), so the number in the JSON line and the capture
# it came from cannot drift apart; `roofline.traffic_source` names the file.
TRAFFIC_PROFILES = {
    ("C5", 8, "bf16"): "profiles/warp_kernel_C5_full_size_dram_traffic.md",
    ("C3", 1, "bf16"): "profiles/warp_kernel_C3_C4_full_set.md",
}


def ncu_traffic(name: str, S: int, io: str):
    """(bytes per launch or None, profile file or None) for the workload's dominant kernel."""
    rel = TRAFFIC_PROFILES.get((name, S, io))
    if rel is None:
        return None, None
    try:
        with open(os.path.join(ROOT, rel)) as fh:
            for line in fh:
                key = f"traffic_bytes_per_launch[{name}/S{S}]"
                if line.strip().startswith(key):
                    return int(line.split("=")[1].strip().replace(" ", "").replace("_", "")), rel
    except OSError:
        pass
    return None, None


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            with open(p) as fh:
                return float(json.load(fh)["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.samples = []
        self.proc = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.cmd = ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}",
                        "--format=csv,noheader,nounits", "-lms", "50"]
        except Exception:
            self.cmd = None

    def start(self):
        if self.cmd is None:
            return
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for s in self.samples:
            parts = [p.strip() for p in s.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "power_w_max": max(power) if power else None, "samples": len(sm)}


# ---------------------------------------------------------------------------------
# one workload on one GPU
# ---------------------------------------------------------------------------------
class DeviceCase:
    """Device (and optionally pinned host) buffers of one workload at one shard
    count, plus the closure that makes the one C-ABI call."""

    def __init__(self, w: W.Workload, S: int, rank: int = 0, host: bool = False, io: str = "bf16",
                 head_dim: int = 0):
        from paper_2608_09160_b200 import binding
        self.binding = binding
        self.w, self.S, self.io, self.head_dim = w, S, io, head_dim
        if head_dim and (S != 1 or io != "bf16"):
            raise SystemExit("--head-dim needs --shards 1 and bf16")
        make = W.make_inputs if io == "bf16" else W.make_inputs_e4m3
        inp = make(rank_workload(w, rank))
        if S == 1:
            host_parts = {"q": [inp["q"]], "k": [inp["k"]], "gq": [inp["gamma_q"]], "gk": [inp["gamma_k"]]}
        else:
            host_parts = {"q": W.shard_columns(inp["q"], S), "k": W.shard_columns(inp["k"], S),
                          "gq": W.shard_columns(inp["gamma_q"], S), "gk": W.shard_columns(inp["gamma_k"], S)}
        del inp
        self.dev = {k: [t.cuda() for t in v] for k, v in host_parts.items()}
        if w.in_place:
            self.out_q, self.out_k = self.dev["q"], self.dev["k"]
        else:
            self.out_q = [torch.empty_like(t) for t in self.dev["q"]]
            self.out_k = [torch.empty_like(t) for t in self.dev["k"]]
        self.host_src = {k: host_parts[k] for k in ("q", "k")} if host else None   # staged by prepare_e2e
        # every element read once and written once (1 or 2 bytes), every gamma (bf16) read once
        eb = 2 if io == "bf16" else 1
        self.bytes = 2 * w.tokens * (w.dq + w.dk) * eb + (w.dq + w.dk) * 2
        self._call = None
        self.fwd = binding.qknorm_fwd if io == "bf16" else binding.qknorm_fwd_e4m3
        self.fwd_sharded = binding.qknorm_fwd_sharded if io == "bf16" else binding.qknorm_fwd_sharded_e4m3

    def _prepared(self, q, k, oq, ok):
        """The one C-ABI call for these buffers with its arguments marshalled once, so that the
        timed loops measure the library and the GPU, not Python argument checking."""
        b, d = self.binding, self.dev
        if self.head_dim:
            return b.prepared(b.qknorm_fwd_headwise, q[0], k[0], d["gq"][0], d["gk"][0], self.head_dim, self.w.eps,
                              oq[0], ok[0])
        if self.S == 1:
            return b.prepared(self.fwd, q[0], k[0], d["gq"][0], d["gk"][0], self.w.eps, oq[0], ok[0])
        return b.prepared(self.fwd_sharded, q, k, d["gq"], d["gk"], self.w.eps, oq, ok)

    def call(self):
        if self._call is None:
            self._call = self._prepared(self.dev["q"], self.dev["k"], self.out_q, self.out_k)
        self._call()

    def prepare_e2e(self, nchunks: int = 32):
        """Cuts the step into token chunks so that the copy engines run in both directions
        while the kernel works: chunk i+1 comes in and chunk i-1 goes out while chunk i is
        normalised.  A chunk's rows of every slice lie back to back in ONE pinned host buffer and
        in one device buffer of the same layout, so a chunk crosses PCIe as one copy per direction
        (with one copy per slice, 16 per chunk here, the copies' own set-up costs 2 ms of a 28 ms
        step); the C-ABI call of the chunk gets the slices as views into that device buffer."""
        T = self.w.tokens
        if T < 8 * 1024:
            nchunks = 1
        edges = [T * i // nchunks for i in range(nchunks + 1)]
        self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
        self.chunks = []
        parts = [(n, i) for n in ("q", "k") for i in range(len(self.host_src[n]))]
        for t0, t1 in zip(edges[:-1], edges[1:]):
            rows = t1 - t0
            sizes = [rows * self.host_src[n][i].shape[1] for n, i in parts]
            total = sum(sizes)
            dtype = self.host_src["q"][0].dtype
            h_in, h_out = torch.empty(total, dtype=dtype).pin_memory(), torch.empty(total, dtype=dtype).pin_memory()
            d_in = torch.empty(total, dtype=dtype, device="cuda")
            d_out = d_in if self.w.in_place else torch.empty_like(d_in)
            views = {"q": [], "k": []}
            outs = {"q": [], "k": []}
            off = 0
            for (n, i), size in zip(parts, sizes):
                src = self.host_src[n][i][t0:t1]
                h_in[off:off + size].view(rows, -1).copy_(src)
                views[n].append(d_in[off:off + size].view(rows, -1))
                outs[n].append(d_out[off:off + size].view(rows, -1))
                off += size
            self.chunks.append({"h_in": h_in, "h_out": h_out, "d_in": d_in, "d_out": d_out,
                                "call": self._prepared(views["q"], views["k"], outs["q"], outs["k"])})
        return nchunks

    def e2e_step(self):
        """Inputs from pinned host memory, the call(s), the result back to pinned host memory."""
        cur = torch.cuda.current_stream()
        self.s_in.wait_stream(cur)
        self.s_out.wait_stream(cur)
        for c in self.chunks:
            with torch.cuda.stream(self.s_in):
                c["d_in"].copy_(c["h_in"], non_blocking=True)
                ev_in = self.s_in.record_event()
            cur.wait_event(ev_in)
            c["call"]()
            self.s_out.wait_event(cur.record_event())
            with torch.cuda.stream(self.s_out):
                c["h_out"].copy_(c["d_out"], non_blocking=True)
        cur.wait_stream(self.s_out)

    def e2e_bytes(self):
        n = sum(c["h_in"].numel() * c["h_in"].element_size() for c in self.chunks)
        return n, n


def time_calls(fn, steps: int, warmup: int):
    """Per-call device times (ms) with CUDA events on the current stream."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def time_region(fn, steps: int):
    """Total device time (ms) of `steps` back-to-back calls."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b)


def graph_replay_us(case: DeviceCase, calls_per_graph: int = 50, replays: int = 20) -> float:
    """us per call when `calls_per_graph` calls are captured in one CUDA graph and replayed."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for _ in range(3):
            case.call()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(calls_per_graph):
            case.call()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(replays):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b) * 1e3 / calls_per_graph)
    return statistics.median(ts)


def graph_replay_cold_us(case: DeviceCase, replays: int = 10) -> float:
    """us per call with the call's data NOT in L2: one CUDA graph of K calls, each on its own copy of
    the buffers, K chosen so that the copies together are more than twice the 126 MB L2; by the time a
    replay comes back to a copy, everything the graph touched since has pushed it out."""
    sets = max(4, int(2.2 * L2_BYTES / max(case.bytes, 1)) + 1)
    dev = case.dev

    def clones(ts):
        return [[t.clone() for t in ts] for _ in range(sets)]
    qs, ks = clones(dev["q"]), clones(dev["k"])
    oqs = qs if case.w.in_place else clones(dev["q"])
    oks = ks if case.w.in_place else clones(dev["k"])
    calls = [case._prepared(qs[i], ks[i], oqs[i], oks[i]) for i in range(sets)]
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        calls[0]()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for c in calls:
            c()
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(replays):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b) * 1e3 / sets)
    return statistics.median(ts)


def copy_rate_same_bytes(nbytes: int, steps: int = 10) -> float:
    """GB/s (read + write bytes) of a device-to-device copy that moves the same number of
    bytes as one call: what a plain memcpy of this size reaches on this GPU, ramp-up included."""
    n = max(nbytes // 4, 1)                      # int16 elements: n*2 bytes read + n*2 bytes written
    a = torch.empty((n,), dtype=torch.int16, device="cuda")
    b = torch.empty_like(a)
    ts = time_calls(lambda: b.copy_(a), steps, 3)
    del a, b
    return 4 * n / (statistics.median(ts) * 1e-3) / 1e9


def config_table(steps: int, warmup: int, peak: float, skip: str, scope: str = "all"):
    """us/call, GB/s and roofline fraction of every workload other than the headline one."""
    from paper_2608_09160_b200 import binding
    rows = {}
    todo = [(name, S, "bf16") for name, w in W.WORKLOADS.items() for S in w.shards]
    if scope == "all":
        # FP8-E4M3 activations (Section IV-C), the prefill workloads at their last shard count
        todo += [(name, W.WORKLOADS[name].shards[-1], "e4m3") for name in ("C3", "C4", "C5")]
    for name, S, io in todo:
        w = W.WORKLOADS[name]
        key = f"{name}/S{S}" + ("" if io == "bf16" else "/e4m3")
        if key == skip:
            continue
        case = DeviceCase(w, S, io=io)
        ts = time_calls(case.call, max(steps, 10), max(warmup, 3))
        med, mn = statistics.median(ts), min(ts)
        torch.cuda.synchronize()
        b2b = time_region(case.call, max(steps, 10)) / max(steps, 10)
        row = {"us_median": round(med * 1e3, 3), "us_min": round(mn * 1e3, 3),
               "us_back_to_back": round(b2b * 1e3, 3),
               "GBps": round(case.bytes / (med * 1e-3) / 1e9, 1),
               "GBps_back_to_back": round(case.bytes / (b2b * 1e-3) / 1e9, 1),
               "frac_measured_peak_back_to_back": round(case.bytes / (b2b * 1e-3) / 1e9 / peak, 4),
               "frac_measured_peak": round(case.bytes / (med * 1e-3) / 1e9 / peak, 4),
               "frac_nominal_8TBps": round(case.bytes / (med * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
               "bytes": case.bytes, "variant": binding.last_variant(),
               "l2": "resident (working set < L2)" if case.bytes < 100e6 else "inputs larger than L2",
               "same_size_copy_GBps": None}
        if w.tokens <= 1024:
            row["us_graph_replay"] = round(graph_replay_us(case), 3)            # L2-warm, launch amortised
            row["us_graph_replay_l2_cold"] = round(graph_replay_cold_us(case), 3)  # every call on data not in L2
        else:
            row["same_size_copy_GBps"] = round(copy_rate_same_bytes(case.bytes), 1)
        rows[key] = row
        del case
        torch.cuda.empty_cache()
    if scope == "all":
        rows.update(variant_rows(steps, warmup, peak))
        rows.update(baseline_rows(steps, warmup, peak))
        rows.update(tp_rows(steps, warmup, peak))
    return rows


def per_config_summary(table: dict, headline_key: str, headline_row: dict) -> dict:
    """The five workloads of the metric at their shard counts, one compact row each (time of an
    isolated call, time per call back to back, GB/s and fraction of the measured copy rate from the
    back-to-back time, kernel variant; decode sizes: CUDA-graph replay with the data in L2 and not)."""
    out = {headline_key: headline_row}
    for name, w in W.WORKLOADS.items():
        for S in w.shards:
            key = f"{name}/S{S}"
            r = table.get(key)
            if r is None:
                continue
            row = {"us_median": r["us_median"], "us_back_to_back": r["us_back_to_back"], "variant": r["variant"]}
            if "us_graph_replay" in r:
                row["us_graph_replay"] = r["us_graph_replay"]
                row["us_graph_replay_l2_cold"] = r["us_graph_replay_l2_cold"]
            else:
                row["GBps"] = r["GBps_back_to_back"]
                row["frac"] = r["frac_measured_peak_back_to_back"]
                row["frac_isolated_median"] = r["frac_measured_peak"]
            out[key] = row
    return dict(sorted(out.items()))


def tp_rows(steps: int, warmup: int, peak: float, tokens: int = 0):
    """The tensor-parallel kernel (Algorithm 1 with its scalar exchange) with all N ranks on this
    one GPU: one cooperative launch serves every rank, scalars go through the ranks' inboxes in
    device memory.  Same bytes as the logical-shard call, so the difference to it is what the
    exchange protocol itself costs when the link is free."""
    from paper_2608_09160_b200 import binding, tp
    rows = {}
    for name, N in (("C3", 4), ("C4", 8), ("C5", 8)):
        w = W.WORKLOADS[name] if tokens <= 0 else W.scaled(W.WORKLOADS[name], tokens)
        inp = W.make_inputs(w)
        dev = {k: [t.cuda() for t in W.shard_columns(inp[k], N)] for k in ("q", "k", "gamma_q", "gamma_k")}
        del inp
        grp = tp.EmulatedGroup(N, token_capacity=w.tokens)
        bufs = grp.buffers(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], out_q=dev["q"], out_k=dev["k"])
        call = grp.prepare(bufs, w.eps)
        ts = time_calls(lambda: call(grp.epochs.next()), max(steps, 10), max(warmup, 3))
        med = statistics.median(ts)
        gbs = w.algorithmic_bytes / (med * 1e-3) / 1e9
        ok = all(tp.status(b)["status"] == tp.STATUS_OK for b in grp.inboxes)
        rows[f"{name}/TP{N}-one-GPU-emulation/in-place"] = {
            "us_median": round(med * 1e3, 3), "us_min": round(min(ts) * 1e3, 3), "GBps": round(gbs, 1),
            "frac_measured_peak": round(gbs / peak, 4), "frac_nominal_8TBps": round(gbs / NOMINAL_HBM_GBS, 4),
            "bytes": w.algorithmic_bytes, "variant": binding.last_variant(), "l2": "inputs larger than L2",
            "exchange_bytes_per_call": 16 * w.tokens * N * (N - 1), "all_waits_completed": ok}
        del dev, bufs, call, grp
        torch.cuda.empty_cache()
    return rows


def baseline_rows(steps: int, warmup: int, peak: float):
    """The one-GPU stand-ins for the paper's comparison paths on the sharded prefill workloads,
    next to the fused call on the same buffers: time and time relative to fused (the
    paper's Fig. 3a normalises latency the same way).  GB/s counts the ALGORITHMIC bytes
    of the fused op, so the stand-ins' extra traffic shows up as a lower figure."""
    from paper_2608_09160_b200 import binding
    rows = {}
    for name in ("C4", "C5"):
        w = W.WORKLOADS[name]
        S = w.shards[-1]
        case = DeviceCase(w, S)
        d = case.dev
        scratch_g = torch.empty((w.tokens * (w.dq + w.dk),), dtype=torch.bfloat16, device="cuda")
        scratch_s = torch.empty((2 * S * w.tokens,), dtype=torch.float32, device="cuda")
        calls = {
            "fused": case.call,
            "baseline-gather-then-norm": binding.prepared(
                binding.qknorm_baseline_gather_then_norm, d["q"], d["k"], d["gq"], d["gk"], w.eps, case.out_q,
                case.out_k, scratch=scratch_g),
            "baseline-two-pass": binding.prepared(
                binding.qknorm_baseline_two_pass, d["q"], d["k"], d["gq"], d["gk"], w.eps, case.out_q, case.out_k,
                scratch=scratch_s),
        }
        med = {}
        for key, fn in calls.items():
            ts = time_calls(fn, max(steps, 10), max(warmup, 3))
            med[key] = statistics.median(ts)
        for key in ("baseline-gather-then-norm", "baseline-two-pass"):
            gbs = case.bytes / (med[key] * 1e-3) / 1e9
            rows[f"{name}/S{S}/{key}"] = {
                "us_median": round(med[key] * 1e3, 3), "GBps": round(gbs, 1), "frac_measured_peak": round(gbs / peak, 4),
                "fused_us_same_buffers": round(med["fused"] * 1e3, 3),
                "time_relative_to_fused": round(med[key] / med["fused"], 3),
                "launches_per_call": 2, "bytes": case.bytes, "variant": "baseline"}
        del case, scratch_g, scratch_s, d
        torch.cuda.empty_cache()
    # The paper's own token counts (Fig. 3a: 64 and 4096 input tokens) on the C3 and C4 shapes, each
    # call timed under CUDA-graph replay (these calls are short): the fused call's latency as a
    # fraction of each stand-in's, the form in which Section IV-B quotes its latency reductions.
    for name, S in (("C3", 4), ("C4", 8)):
        for tokens in (64, 4096):
            w = W.scaled(W.WORKLOADS[name], tokens)
            case = DeviceCase(w, S)
            d = case.dev
            scratch_g = torch.empty((w.tokens * (w.dq + w.dk),), dtype=torch.bfloat16, device="cuda")
            scratch_s = torch.empty((2 * S * w.tokens,), dtype=torch.float32, device="cuda")
            calls = {
                "fused": case.call,
                "baseline-gather-then-norm": binding.prepared(
                    binding.qknorm_baseline_gather_then_norm, d["q"], d["k"], d["gq"], d["gk"], w.eps, case.out_q,
                    case.out_k, scratch=scratch_g),
                "baseline-two-pass": binding.prepared(
                    binding.qknorm_baseline_two_pass, d["q"], d["k"], d["gq"], d["gk"], w.eps, case.out_q, case.out_k,
                    scratch=scratch_s),
            }
            us = {}
            for key, fn in calls.items():
                holder = type("Call", (), {"call": staticmethod(fn)})
                us[key] = graph_replay_us(holder, calls_per_graph=20, replays=10)
            rows[f"{name}/S{S}/T{tokens}/latency-vs-stand-ins"] = {
                "fused_us": round(us["fused"], 3),
                "gather_then_norm_us": round(us["baseline-gather-then-norm"], 3),
                "two_pass_us": round(us["baseline-two-pass"], 3),
                "latency_reduction_vs_gather_then_norm_pct": round(100 * (1 - us["fused"] / us["baseline-gather-then-norm"]), 1),
                "latency_reduction_vs_two_pass_pct": round(100 * (1 - us["fused"] / us["baseline-two-pass"]), 1),
                "how": "CUDA-graph replay of 20 calls on the same buffers (in L2 at 64 tokens; 100-170 MB at 4096)",
                "variant": "baseline"}
            del case, scratch_g, scratch_s, d
            torch.cuda.empty_cache()
    return rows


def variant_rows(steps: int, warmup: int, peak: float):
    """The two layout/granularity variants on the C4 and C5 shapes (unsharded, bf16):
    rows strided inside a fused [T, dq + 2*dk] projection output, and headwise (head_dim 128)."""
    from paper_2608_09160_b200 import binding
    rows = {}
    for name in ("C4", "C5"):
        w = W.WORKLOADS[name]
        inp = W.make_inputs(w)
        gq, gk = inp["gamma_q"].cuda(), inp["gamma_k"].cuda()
        buf = torch.empty((w.tokens, w.dq + 2 * w.dk), dtype=torch.bfloat16, device="cuda")
        buf[:, :w.dq] = inp["q"].cuda()
        buf[:, w.dq:w.dq + w.dk] = inp["k"].cuda()
        del inp
        q, k = buf[:, :w.dq], buf[:, w.dq:w.dq + w.dk]
        calls = {
            f"{name}/fusedQKV-strided/in-place": binding.prepared(binding.qknorm_fwd_strided, q, k, gq, gk, w.eps),
            f"{name}/headwise128/fusedQKV/in-place": binding.prepared(binding.qknorm_fwd_headwise, q, k, gq, gk, 128,
                                                                      w.eps, q, k),
        }
        for key, fn in calls.items():
            ts = time_calls(fn, max(steps, 10), max(warmup, 3))
            med = statistics.median(ts)
            gbs = w.algorithmic_bytes / (med * 1e-3) / 1e9
            rows[key] = {"us_median": round(med * 1e3, 3), "us_min": round(min(ts) * 1e3, 3), "GBps": round(gbs, 1),
                         "frac_measured_peak": round(gbs / peak, 4), "frac_nominal_8TBps": round(gbs / NOMINAL_HBM_GBS, 4),
                         "bytes": w.algorithmic_bytes, "variant": binding.last_variant(), "l2": "inputs larger than L2"}
        del buf, q, k
        torch.cuda.empty_cache()
    # headwise on the C5 shape as 8 column slices in one launch (bf16), and on whole FP8-E4M3 rows
    w = W.WORKLOADS["C5"]
    for key, io in ((f"C5/headwise128/S8-one-launch/in-place", "bf16"), ("C5/headwise128/e4m3/in-place", "e4m3")):
        inp = (W.make_inputs if io == "bf16" else W.make_inputs_e4m3)(w)
        eb = 2 if io == "bf16" else 1
        nbytes = 2 * w.tokens * (w.dq + w.dk) * eb + (w.dq + w.dk) * 2
        if io == "bf16":
            d = {n: [t.cuda() for t in W.shard_columns(inp[n], 8)] for n in ("q", "k", "gamma_q", "gamma_k")}
            fn = binding.prepared(binding.qknorm_fwd_headwise_sharded, d["q"], d["k"], d["gamma_q"], d["gamma_k"], 128,
                                  w.eps, d["q"], d["k"])
        else:
            d = {n: inp[n].cuda() for n in ("q", "k", "gamma_q", "gamma_k")}
            fn = binding.prepared(binding.qknorm_fwd_headwise_e4m3, d["q"], d["k"], d["gamma_q"], d["gamma_k"], 128,
                                  w.eps, d["q"], d["k"])
        del inp
        ts = time_calls(fn, max(steps, 10), max(warmup, 3))
        med = statistics.median(ts)
        gbs = nbytes / (med * 1e-3) / 1e9
        rows[key] = {"us_median": round(med * 1e3, 3), "us_min": round(min(ts) * 1e3, 3), "GBps": round(gbs, 1),
                     "frac_measured_peak": round(gbs / peak, 4), "frac_nominal_8TBps": round(gbs / NOMINAL_HBM_GBS, 4),
                     "bytes": nbytes, "variant": binding.last_variant(), "l2": "inputs larger than L2"}
        del d, fn
        torch.cuda.empty_cache()
    # short rows: what ONE of 8 tensor-parallel ranks holds of C5 (its column slice), normalised on
    # its own as unsharded rows -- the shape the tiled kernel exists for
    w = W.Workload("C5-slice", tokens=65536, dq=1024, dk=128, shards=(1,), sigma=2.0, seed=4, in_place=True)
    case = DeviceCase(w, 1)
    ts = time_calls(case.call, max(steps, 10), max(warmup, 3))
    med = statistics.median(ts)
    gbs = case.bytes / (med * 1e-3) / 1e9
    rows["C5-one-rank-slice(1024+128)/unsharded/in-place"] = {
        "us_median": round(med * 1e3, 3), "us_min": round(min(ts) * 1e3, 3), "GBps": round(gbs, 1),
        "frac_measured_peak": round(gbs / peak, 4), "frac_nominal_8TBps": round(gbs / NOMINAL_HBM_GBS, 4),
        "bytes": case.bytes, "variant": binding.last_variant(), "l2": "inputs larger than L2",
        "same_size_copy_GBps": round(copy_rate_same_bytes(case.bytes), 1)}
    del case
    torch.cuda.empty_cache()
    return rows


# ---------------------------------------------------------------------------------
# the CPU oracle, timed
# ---------------------------------------------------------------------------------
def oracle_sample_inputs(w: W.Workload, tokens: int):
    import numpy as np  # noqa: F401
    ws = W.scaled(w, tokens)
    inp = W.make_inputs(ws)
    return ws, {k: W.bf16_bits(v) for k, v in inp.items()}


def run_oracle_once(bits, eps, nthreads):
    import oracle
    t0 = time.perf_counter()
    oracle.rmsnorm(bits["q"], bits["gamma_q"], eps, nthreads=nthreads)
    oracle.rmsnorm(bits["k"], bits["gamma_k"], eps, nthreads=nthreads)
    return time.perf_counter() - t0


def cpu_baseline(w: W.Workload, target_cpu_seconds: float = 16.0):
    """Times the oracle on a bounded sample (first `n` tokens' worth of the same
    recipe) with all host cores; sized so that it costs ~10-30 s of CPU work."""
    import oracle
    cores = min(os.cpu_count() or 1, oracle.max_threads())
    ws, bits = oracle_sample_inputs(w, 256)
    run_oracle_once(bits, w.eps, cores)                       # warm (builds/loads the library)
    dt = run_oracle_once(bits, w.eps, cores)
    cpu_s_per_token = dt * cores / 256
    n = int(max(256, min(w.tokens, target_cpu_seconds / max(cpu_s_per_token, 1e-9))))
    ws, bits = oracle_sample_inputs(w, n)
    dt = run_oracle_once(bits, w.eps, cores)
    gbs = ws.algorithmic_bytes / dt / 1e9
    # the same oracle on ONE thread, on a sample 1/cores as long (about a second)
    n1 = max(64, n // max(cores, 1))
    ws1, bits1 = oracle_sample_inputs(w, n1)
    dt1 = run_oracle_once(bits1, w.eps, 1)
    return {"value": round(gbs, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} of {w.tokens} tokens of {w.name} (dq={w.dq}, dk={w.dk}), "
                      f"unsharded definition, one pass, {dt:.2f} s wall",
            "seconds": round(dt, 3),
            "single_thread": {"value": round(ws1.algorithmic_bytes / dt1 / 1e9, 4), "unit": UNIT, "cores": 1,
                              "sample": f"first {n1} tokens, one pass, {dt1:.2f} s wall"}}


def rank_workload(w: W.Workload, rank: int) -> W.Workload:
    """The path shards by token range with no exchange: rank r normalises its own tokens.
    Weak scaling: every rank gets the workload's shape with its own seed (its own tokens)."""
    return W.Workload(**{**w.__dict__, "seed": w.seed + 1000 * rank})


def max_over_ranks(ms: float, dist, device) -> float:
    """Job time = the slowest rank's device time (all_reduce MAX); identity on one rank."""
    if dist is None:
        return ms
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(bytes_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job GB/s: the bytes all ranks processed in the time the slowest one took."""
    return world * bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def case_bytes_of(w: W.Workload, io: str) -> int:
    eb = 2 if io == "bf16" else 1
    return 2 * w.tokens * (w.dq + w.dk) * eb + (w.dq + w.dk) * 2


def config_of(w: W.Workload, S: int, world: int, variant=None, io: str = "bf16", head_dim: int = 0):
    """The `config` object of the JSON line (the same for both arms)."""
    cfg = {"workload": f"{w.name}: {w.note}", "tokens": w.tokens, "dq": w.dq, "dk": w.dk, "num_shards": S,
           "in_place": w.in_place, "storage": io, "eps": w.eps,
           "granularity": f"headwise, head_dim {head_dim}" if head_dim else "layerwise",
           "bytes_per_step_per_gpu": case_bytes_of(w, io),
           "parallelism": f"token-range x{world}, no collective",
           "l2": "inputs larger than L2 (no flush needed)" if w.algorithmic_bytes > 300e6
                 else "working set fits in L2 (L2-warm number)"}
    if variant is not None:
        cfg["kernel_variant"] = variant
    return cfg


# ---------------------------------------------------------------------------------
# column-sharded mode: one rank per GPU, Algorithm 1's scalar exchange between the GPUs
# ---------------------------------------------------------------------------------
def tp_rank_inputs(w: W.Workload, world: int, rank: int, io: str = "bf16"):
    """Rank `rank`'s column slice of the workload (every rank draws the same full tensors from the
    workload's seed and keeps its own slice: what a column-parallel projection leaves on the rank)."""
    inp = (W.make_inputs if io == "bf16" else W.make_inputs_e4m3)(w)
    return {n: W.shard_columns(inp[n], world)[rank].contiguous() for n in ("q", "k", "gamma_q", "gamma_k")}


def run_tp_parallel(w: W.Workload, world: int, rank: int, dist, steps: int, warmup: int, *, device="cuda",
                    io: str = "bf16", ipc=None, launch=None, e2e: bool = False):
    """The timed region of `--parallelism tp`: every rank holds its column slice, the communicator
    wires the inboxes, and a step is one `comm.forward` (one launch per rank; the ranks' kernels
    push their partial sums of squares into each other's inboxes).  Returns this rank's record with
    the job time already the MAX over ranks.  `ipc` / `launch` are the communicator's stand-ins
    (tests on CPU); with them nothing here touches CUDA."""
    from paper_2608_09160_b200 import tp
    on_gpu = device != "cpu"
    host = tp_rank_inputs(w, world, rank, io)
    dev = {n: t.to(device) for n, t in host.items()}
    out_q = dev["q"] if w.in_place else torch.empty_like(dev["q"])
    out_k = dev["k"] if w.in_place else torch.empty_like(dev["k"])
    comm = tp.Communicator(w.tokens, ipc=ipc, launch=launch)
    bufs = comm.buffers(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], out_q=out_q, out_k=out_k)
    prepared = comm.prepare(bufs, w.eps) if launch is None else None

    def step():
        comm.forward(bufs, w.eps, prepared=prepared)

    def barrier():
        dist.barrier()
        if on_gpu:
            torch.cuda.synchronize()

    def timed(fn, n):
        barrier()
        if on_gpu:
            ms = time_region(fn, n)
        else:
            t0 = time.perf_counter()
            for _ in range(n):
                fn()
            ms = (time.perf_counter() - t0) * 1e3
        barrier()
        return max_over_ranks(ms, dist if world > 1 else None, device)

    for _ in range(warmup):
        step()
    first_epoch = comm.epochs.last
    if launch is None:
        from paper_2608_09160_b200 import binding
        n0 = binding.launch_count()
    total_ms = timed(step, steps)
    rec = {"ms_per_step": total_ms / steps, "epochs": (first_epoch, comm.epochs.last),
           "launches": (binding.launch_count() - n0) if launch is None else 0,
           "variant": binding.last_variant() if launch is None else None,
           "rank_bytes": 2 * w.tokens * (dev["q"].shape[1] + dev["k"].shape[1]) * dev["q"].element_size()
                         + (dev["q"].shape[1] + dev["k"].shape[1]) * 2,
           "job_bytes": case_bytes_of(w, io), "e2e": None}
    if e2e and on_gpu:
        pin = {n: host[n].pin_memory() for n in ("q", "k")}
        back = {n: torch.empty_like(pin[n]).pin_memory() for n in ("q", "k")}

        def e2e_step():
            dev["q"].copy_(pin["q"], non_blocking=True)
            dev["k"].copy_(pin["k"], non_blocking=True)
            step()
            back["q"].copy_(out_q, non_blocking=True)
            back["k"].copy_(out_k, non_blocking=True)
        e2e_step()
        e_ms = timed(e2e_step, steps)
        nbytes = sum(pin[n].numel() * pin[n].element_size() for n in ("q", "k"))
        rec["e2e"] = {"ms_per_step": e_ms / steps, "h2d": nbytes, "d2h": nbytes}
    rec["status"] = comm.status()
    comm.close()
    return rec


def tp_line(w: W.Workload, world: int, args, rec: dict, peak: float, peak_kind: str, variant, launches: int, clocks):
    """The contract line of `--parallelism tp` (rank 0 prints it)."""
    ms = rec["ms_per_step"]
    value = rec["job_bytes"] / (ms * 1e-3) / 1e9                 # all ranks' bytes over the slowest rank's time
    per_gpu = rec["rank_bytes"] / (ms * 1e-3) / 1e9
    cfg = config_of(w, world, world, variant, args.dtype)
    cfg["parallelism"] = f"tensor-parallel x{world}, scalar exchange"
    cfg["bytes_per_step_per_gpu"] = rec["rank_bytes"]
    e2e = None
    if rec["e2e"] is not None:
        e = rec["e2e"]
        e2e = {"value": round(rec["job_bytes"] / (e["ms_per_step"] * 1e-3) / 1e9, 3), "unit": UNIT,
               "h2d_bytes_per_step": e["h2d"], "d2h_bytes_per_step": e["d2h"], "ms_per_step": round(e["ms_per_step"], 3),
               "how": "per rank: the slice from pinned host memory, one call, the slice back to pinned host memory"}
    return {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms, 5), "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None, "dtype": "f32", "storage_dtype": args.dtype, "accum_dtype": "f32",
        "data": "synthetic", "config": cfg, "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": round(per_gpu, 1), "peak": peak, "unit": UNIT,
                     "frac": round(per_gpu / peak, 4), "traffic": None, "peak_kind": f"{peak_kind} device copy rate (hbm_gbs)",
                     "per_gpu": True, "kernel_variant": variant,
                     "exchange_bytes_per_step_per_gpu": 16 * w.tokens * (world - 1),
                     "all_waits_completed": rec["status"].get("status") == 0},
        "cpu_baseline": None,
    }


def run_reference(args):
    """--impl reference: the oracle as it stands, on host cores, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    w = W.WORKLOADS[args.workload]
    if args.tokens:
        w = W.scaled(w, args.tokens)
    S = args.shards or w.shards[0]
    cores = min(os.cpu_count() or 1, oracle.max_threads())
    ws, bits = oracle_sample_inputs(w, 256)
    run_oracle_once(bits, w.eps, cores)
    dt = run_oracle_once(bits, w.eps, cores)
    # each step about 1.5 s of wall time, bounded by the workload itself
    n = int(max(64, min(w.tokens, 256 * 1.5 / max(dt, 1e-9))))
    ws, bits = oracle_sample_inputs(w, n)
    for _ in range(args.warmup):
        run_oracle_once(bits, w.eps, cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run_oracle_once(bits, w.eps, cores)
    total = time.perf_counter() - t0
    gbs = ws.algorithmic_bytes * args.steps / total / 1e9
    sample = f"each step = first {n} of {w.tokens} tokens of {w.name} (dq={w.dq}, dk={w.dk}), fp64 oracle"
    line = {
        "impl": "reference", "metric": METRIC, "value": round(gbs, 4), "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(total / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, S, 1),
        "cpu_baseline": {"value": round(gbs, 4), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                         "sample_tokens_per_step": n},
        "e2e": {"value": round(gbs, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ---------------------------------------------------------------------------------
# main
# ---------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C5", choices=sorted(W.WORKLOADS))
    ap.add_argument("--shards", type=int, default=0, help="shard count (default: the workload's first)")
    ap.add_argument("--tokens", type=int, default=0, help="override the token count (for profiling a small case)")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "e4m3"], help="storage format of the activations")
    ap.add_argument("--head-dim", type=int, default=0, help="headwise granularity with this head size (needs --shards 1)")
    ap.add_argument("--one-rank-slice", type=int, default=0,
                    help="time the column slice one of N tensor-parallel ranks holds, as unsharded rows (short rows)")
    ap.add_argument("--no-table", action="store_true", help="skip the per-config table")
    ap.add_argument("--table-scope", default="all", choices=["all", "configs"],
                    help="configs: only the five workloads of the metric; all: also the FP8, strided, headwise, "
                         "short-row, stand-in and tensor-parallel rows")
    ap.add_argument("--tp-only", action="store_true",
                    help="only the tensor-parallel rows of the table (all ranks on this GPU), as one JSON object; "
                         "with --tokens for a small case to profile")
    ap.add_argument("--parallelism", default="tokens", choices=["tokens", "tp"],
                    help="tokens: every GPU normalises its own token range, no exchange (default); "
                         "tp: every GPU holds a column slice and the GPUs exchange Algorithm 1's scalars")
    ap.add_argument("--configs-out", default="", help="also write the full per-config table to this JSON file")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-chunks", type=int, default=32, help="token chunks of the host-to-host pipeline")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        log("note: fewer than 3 warm-up steps requested")

    if args.impl == "reference":
        return run_reference(args)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2608_09160_b200 import binding, build
    if rank == 0:
        build.build()
    if dist is not None:
        dist.barrier()
    binding.load()
    if args.tp_only:
        if world > 1:
            raise SystemExit("--tp-only stands N ranks on ONE GPU; run it without torchrun")
        print(json.dumps({"tensor_parallel_rows": tp_rows(args.steps, args.warmup, measured_peak()[0], args.tokens)}))
        return

    w = W.WORKLOADS[args.workload]
    if args.tokens:
        w = W.scaled(w, args.tokens)
    if args.parallelism == "tp":
        own_group = dist is None
        if own_group:     # one rank: the communicator still wants a process group for its host-side exchange
            import socket
            import torch.distributed as dist
            with socket.socket() as sock:
                sock.bind(("127.0.0.1", 0))
                port = sock.getsockname()[1]
            dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
        peak, peak_kind = measured_peak()
        sampler = ClockSampler(local)
        sampler.start()
        rec = run_tp_parallel(w, world, rank, dist, args.steps, args.warmup, io=args.dtype, e2e=not args.no_e2e)
        clocks = sampler.stop()
        if rank == 0:
            print(json.dumps(tp_line(w, world, args, rec, peak, peak_kind, rec["variant"], rec["launches"], clocks)),
                  flush=True)
        dist.destroy_process_group()
        return 0
    S = args.shards or w.shards[0]
    if args.one_rank_slice:
        # what ONE of n tensor-parallel ranks holds of the workload (its column slice), as unsharded rows
        n = args.one_rank_slice
        w = dataclasses.replace(w, name=f"{w.name}-slice-of-{n}", dq=w.dq // n, dk=w.dk // n, shards=(1,),
                                note=f"column slice of one of {n} ranks, unsharded")
        S = 1
    peak, peak_kind = measured_peak()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    case = DeviceCase(w, S, rank=rank, host=not args.no_e2e, io=args.dtype, head_dim=args.head_dim)

    # ---- device-resident timing -----------------------------------------------------------
    for _ in range(args.warmup):
        case.call()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    per_call = time_calls(case.call, args.steps, 0)          # one event pair per launch (roofline.achieved)
    barrier()
    n0 = binding.launch_count()
    total_ms = time_region(case.call, args.steps)            # THE timed region: K steps, back to back
    barrier()
    launches = binding.launch_count() - n0                   # kernels of this library launched inside it
    variant = binding.last_variant()                         # the kernel the timed launches ran
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    ms_per_step = total_ms / args.steps
    value = job_value(case.bytes, world, ms_per_step)
    # the kernel's average launch duration over the timed region (one launch per step on this GPU)
    launch_ms = total_ms / max(launches, 1)
    achieved = case.bytes / (launch_ms * 1e-3) / 1e9

    # ---- end to end: host buffers in, host buffers out ----------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e_chunks = case.prepare_e2e(args.e2e_chunks)
        for _ in range(2):
            case.e2e_step()
        barrier()
        e_ms = time_region(case.e2e_step, args.steps)
        barrier()
        e_ms = max_over_ranks(e_ms, dist, "cuda")
        h2d, d2h = case.e2e_bytes()
        e2e = {"value": round(job_value(case.bytes, world, e_ms / args.steps), 3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": round(e_ms / args.steps, 3), "calls_per_step": e2e_chunks,
               "kernel_variant": binding.last_variant(),
               "how": "pinned host buffers -> device -> C-ABI call -> pinned host buffers, in token chunks "
                      "(one copy per chunk and direction) so that both copy directions overlap the kernel"}
    clocks = sampler.stop()      # sampled over the device-resident and the end-to-end timed regions
    del case
    torch.cuda.empty_cache()
    case_bytes = case_bytes_of(w, args.dtype)
    same_size_copy = copy_rate_same_bytes(case_bytes) if rank == 0 else None
    torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    table = None
    if not args.no_table and world == 1:
        table = config_table(args.steps, args.warmup, peak, skip=f"{w.name}/S{S}", scope=args.table_scope)
    cpu = None
    if not args.no_cpu and world == 1:
        cpu = cpu_baseline(w)

    traffic, traffic_source = (ncu_traffic(w.name, S, args.dtype) if not (args.head_dim or args.tokens or args.one_rank_slice)
                               else (None, None))
    isolated_med = statistics.median(per_call)
    roofline = {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": UNIT,
                "frac": round(achieved / peak, 4), "traffic": traffic, "traffic_source": traffic_source,
                "peak_kind": f"{peak_kind} device copy rate (hbm_gbs)",
                "frac_of_nominal_8TBps": round(achieved / NOMINAL_HBM_GBS, 4),
                "algorithmic_bytes_per_launch": case_bytes,
                "same_size_copy_GBps": round(same_size_copy, 1),
                "kernel_variant": variant,
                "how": "achieved = algorithmic bytes per launch / (device time of the timed region / launches in it); "
                       "launches of one stream overlap their start-up with the previous kernel's tail",
                "launch_us_mean": round(launch_ms * 1e3, 3),
                # the same launches timed one by one (an event pair around each, so no overlap between them)
                "launch_us_isolated_median": round(isolated_med * 1e3, 3),
                "launch_us_isolated_min": round(min(per_call) * 1e3, 3),
                "frac_isolated_median": round(case_bytes / (isolated_med * 1e-3) / 1e9 / peak, 4)}
    if table is not None:
        roofline["per_config"] = per_config_summary(table, f"{w.name}/S{S}", {
            "us_median": round(isolated_med * 1e3, 3), "us_back_to_back": round(launch_ms * 1e3, 3),
            "GBps": round(achieved, 1), "frac": round(achieved / peak, 4), "variant": variant})

    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "storage_dtype": args.dtype, "accum_dtype": "f32",
        "data": "synthetic",
        "config": config_of(w, S, world, variant, args.dtype, args.head_dim),
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": cpu,
    }
    if table is not None:
        # the full table goes to stderr (and to --configs-out); the line on stdout stays short enough to be kept whole
        # (its roofline.per_config and roofline.widened_rows carry the figures)
        roofline["widened_rows"] = {k: {kk: r[kk] for kk in ("us_median", "us_back_to_back", "GBps", "frac_measured_peak",
                                                             "frac_measured_peak_back_to_back", "variant",
                                                             "time_relative_to_fused", "fused_us",
                                                             "latency_reduction_vs_gather_then_norm_pct",
                                                             "latency_reduction_vs_two_pass_pct") if kk in r}
                                    for k, r in table.items() if k not in roofline["per_config"]}
        if args.configs_out:
            try:
                os.makedirs(os.path.dirname(os.path.abspath(args.configs_out)), exist_ok=True)
                with open(args.configs_out, "w") as fh:
                    json.dump(table, fh, indent=1)
            except OSError as e:
                log(f"could not write {args.configs_out}: {e}")
        log("configs: " + json.dumps(table))
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
