#!/usr/bin/env python
"""Benchmark of the tree-verification hot path (one B200 per rank).

A step = jet_tree_build -> jet_tree_verify_attn for every layer (each layer has its own KV
buffers, so the K/V stream comes from HBM, not from L2) -> jet_tree_accept -> jet_kv_compact
on the Qwen3-8B-shaped workload (batch 1, 32/8 heads, head_dim 128, prefix 4096, 64-node tree).
The metric is microseconds per layer of a whole step (lower is better).  With N > 1 ranks every
rank verifies its own sequence (no data-path collective: the path shards by sequence).

`--impl reference` times the CPU oracle (test infrastructure, never the product path) on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
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

from jet_inputs import CONFIGS, plant_path  # noqa: E402

METRIC = "tree_verify_us_per_layer"
UNIT = "us/layer"

# DRAM traffic of one tree_attn_kernel launch per workload comes from a small tracked file written from ncu
# captures (bytes per launch, or -- for workloads too large to capture whole -- the ratio DRAM bytes /
# algorithmic bytes of a smaller capture of the same kernel), together with the commit it was captured at.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")
MIN_TIMED_SECONDS = 0.5       # every timed region of the attention launches is repeated up to this length


def ncu_traffic(workload_name, bytes_alg):
    """(traffic bytes per launch or None, note) for the named workload."""
    try:
        table = json.load(open(TRAFFIC_FILE))
    except (OSError, ValueError):
        return None, "no capture on file"
    e = table.get(workload_name)
    if not e:
        return None, "no capture on file"
    note = f"ncu capture at commit {e.get('commit', '?')}: {e.get('source', '')}"
    if "bytes_per_launch" in e:
        return int(e["bytes_per_launch"]), note
    return int(e["ratio_to_algorithmic_bytes"] * bytes_alg), note + " (scaled by the algorithmic bytes)"


def workload(name, budget=None, batch=None):
    """The named configuration; a sweep configuration needs --budget (and --batch if it lists several)."""
    c = dict(CONFIGS[name])
    if "B" not in c:
        if budget is None or budget not in c["budgets"]:
            raise SystemExit(f"config {name} is a sweep: pass --budget, one of {c['budgets']}")
        c["B"] = budget
        c.setdefault("N", 12 if budget > 64 else 8)
    if isinstance(c["batch"], (tuple, list)):
        c["batch"] = batch if batch in c["batch"] else c["batch"][0]
    return c


def attn_algorithmic_bytes(c, seq_lens, n_nodes):
    """K and V prefix + tree K/V + Q in + O out + ancestor mask, per layer (all sequences)."""
    B, Hq, Hkv, D = c["B"], c["Hq"], c["Hkv"], c["D"]
    total = 0
    for L in seq_lens:
        total += 2 * L * Hkv * D * 2 + 2 * B * Hkv * D * 2 + 2 * B * Hq * D * 2 + B * ((B + 31) // 32) * 4
    return total


def attn_algorithmic_flops(c, seq_lens, depths):
    B, Hq, Hkv, D = c["B"], c["Hq"], c["Hkv"], c["D"]
    G = Hq // Hkv
    total = 0
    for L, dep in zip(seq_lens, depths):
        total += 4 * B * Hq * D * L + 4 * G * D * Hkv * int(sum(int(d) + 1 for d in dep if d >= 0))
    return total


class ClockSampler:
    """Samples SM clock and throttle reasons while the timed region runs.

    Reads NVML directly from a thread (every 2 ms, so that a timed region of a few milliseconds still gets
    samples); falls back to polling nvidia-smi where the NVML binding is missing.  Read-only: no setting of
    the GPU is touched."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    REASON_BITS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
                   ("sw_power_cap", 0x4))

    def __init__(self, index, uuid=None):
        self.index, self.uuid = index, uuid
        self.rows, self.proc, self.thread = [], None, None
        self.sm, self.reason_mask, self.sm_max = [], 0, None
        self.stop_flag = threading.Event()
        self.nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            handle = None
            if self.uuid:
                for cand in (f"GPU-{self.uuid}", str(self.uuid)):
                    try:
                        handle = pynvml.nvmlDeviceGetHandleByUUID(cand.encode() if hasattr(cand, "encode") else cand)
                        break
                    except Exception:
                        handle = None
            if handle is None:
                handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            reasons_fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(pynvml, "nvmlDeviceGetCurrentClocksThrottleReasons")
            self.nvml = (pynvml, handle, reasons_fn)
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _poll_nvml(self):
        pynvml, handle, reasons_fn = self.nvml
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(handle, pynvml.NVML_CLOCK_SM)))
                self.reason_mask |= int(reasons_fn(handle))
            except Exception:
                break
            time.sleep(0.002)

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.nvml is not None:
            self.stop_flag.set()
            self.thread.join(timeout=2)
            reasons = [n for n, bit in self.REASON_BITS if self.reason_mask & bit]
            return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.sm_max,
                    "reasons": reasons, "samples": len(self.sm), "source": "nvml"}
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 6 and r[2 + i].lower() == "active" for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm), "source": "nvidia-smi"}


# ------------------------------------------------------------------------------------------------
def plant_hidden(st, b, token, parent, depth, n_nodes, length, rng):
    """The planted path for accept_mode "hidden": the hidden state of every node on the path points along the
    LM-head row of the token that must win there (logit ~ 8 * |row| ~ 10 against ~ N(0, 0.16) for every other
    token), the end node's along a token none of its children carries.  Returns the effective path length."""
    import torch
    B, V = st.B, st.V
    max_depth = int(depth[:n_nodes].max())
    eff = min(length, max_depth)
    cands = [v for v in range(n_nodes) if depth[v] == eff]
    end = int(cands[int(rng.integers(0, len(cands)))])

    def point(row, tok):
        w = st.lm_head[tok].float()
        st.hidden[b * B + row].copy_((8.0 * w / w.norm()).bfloat16())
    u = end
    while parent[u] != -1:
        point(int(parent[u]), int(token[u]))
        u = int(parent[u])
    child_tokens = {int(token[cn]) for cn in range(n_nodes) if parent[cn] == end}
    t = int(rng.integers(0, V))
    while t in child_tokens:
        t = (t + 1) % V
    point(end, t)
    return eff


def build_inputs(c, name, seed, device, score_mode="accum_logp", score_alpha=0.0, tail=False, draft_logits=False,
                 target_hidden=False, d_model=4096):
    """Seeded synthetic step inputs on the device.  Returns (VerifyStep, info dict)."""
    import torch
    from paper_2606_18394_b200.step import VerifyStep

    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    batch, layers = c["batch"], c["layers"]
    B, N, W, V, Hq, Hkv, D = c["B"], c["N"], c["W"], c["V"], c["Hq"], c["Hkv"], c["D"]
    if c.get("paged"):
        rng = np.random.default_rng(seed)
        lo, hi = c["L_range"]
        seq = rng.integers(lo, hi + 1, size=batch).astype(np.int32)
        need = [(int(L) + (max(N + 1, B) if tail else N + 1) + 15) // 16 for L in seq]
        num_pages = sum(need) + 3
        perm = rng.permutation(num_pages)
        max_pages = max(need)
        table = np.full((batch, max_pages), 0, dtype=np.int32)
        pos = 0
        for b, cnt in enumerate(need):
            table[b, :cnt] = perm[pos:pos + cnt]
            pos += cnt
        st = VerifyStep(batch=batch, layers=layers, Hq=Hq, Hkv=Hkv, D=D, B=B, N=N, W=W, V=V,
                        max_seq_len=int(seq.max()), page_size=16, num_pages=num_pages, max_pages=max_pages,
                        device=device, tail=tail)
        st.page_table.copy_(torch.from_numpy(table))
    else:
        seq = np.full(batch, c["L"], dtype=np.int32)
        st = VerifyStep(batch=batch, layers=layers, Hq=Hq, Hkv=Hkv, D=D, B=B, N=N, W=W, V=V,
                        max_seq_len=int(c["L"]), device=device, tail=tail)
    st.seq_len0.copy_(torch.from_numpy(seq))
    for t in (st.q, st.tree_k, st.tree_v):
        t.copy_(torch.randn(t.shape, generator=gen, device=device, dtype=torch.float32))
    for layer in range(layers):      # layer by layer: bounded temporaries
        st.k_cache[layer].copy_(torch.randn(st.k_cache[layer].shape, generator=gen, device=device, dtype=torch.float32))
        st.v_cache[layer].copy_(torch.randn(st.v_cache[layer].shape, generator=gen, device=device, dtype=torch.float32))
    if tail:
        st.place_tree()
    # draft log-probs: log_softmax of N(0, sigma) logits with one confident token per depth (p = 0.7),
    # evaluated in fp64 and rounded to fp32
    for b in range(batch):
        logits = torch.randn((N, V), generator=gen, device=device, dtype=torch.float32).double() * c["sigma_draft"]
        top = torch.randint(0, V, (N,), generator=gen, device=device)
        rest = logits.clone()
        rest[torch.arange(N, device=device), top] = -float("inf")
        logits[torch.arange(N, device=device), top] = np.log(0.7 / 0.3) + torch.logsumexp(rest, dim=1)
        # --draft-input logits: the raw logits themselves (jet_tree_build_logits normalises on the fly)
        st.logp[b].copy_(logits.float() if draft_logits else torch.log_softmax(logits, dim=1).float())
    st.draft_logits = draft_logits
    st.root_token.copy_(torch.arange(batch, device=device, dtype=torch.int32) + 1)
    st.logits.copy_(torch.randn(st.logits.shape, generator=gen, device=device, dtype=torch.float32) * c["sigma_target"])
    # plant the target arg-max along one random path of the tree that jet_tree_build produces
    st.score_mode, st.score_alpha = score_mode, score_alpha
    st.seq_len.copy_(st.seq_len0)
    st.tree_build()
    torch.cuda.synchronize()
    parent, depth, token = st.parent.cpu().numpy(), st.depth.cpu().numpy(), st.token.cpu().numpy()
    n_nodes = st.n_nodes.cpu().numpy()
    rng = np.random.default_rng(seed + 1)
    planted = []
    if target_hidden:
        # the acceptance is fed with final hidden states (N(0,1)) and LM-head weights (N(0, 0.02^2)) instead of logits
        st.enable_lm_head(d_model)
        st.accept_mode = "hidden"
        st.hidden.copy_(torch.randn(st.hidden.shape, generator=gen, device=device, dtype=torch.float32))
        st.lm_head.copy_(torch.randn(st.lm_head.shape, generator=gen, device=device, dtype=torch.float32) * 0.02)
    for b in range(batch):
        want = c.get("plant", int(rng.integers(1, N + 1)))
        if target_hidden:
            planted.append(plant_hidden(st, b, token[b], parent[b], depth[b], int(n_nodes[b]), want, rng))
            continue
        rows = st.logits[b].cpu().numpy()
        _, eff = plant_path(rows, token[b], parent[b], depth[b], int(n_nodes[b]), want, rng)
        st.logits[b].copy_(torch.from_numpy(rows))
        planted.append(eff)
    info = dict(seq_lens=[int(x) for x in seq], planted=planted, depth=depth, n_nodes=n_nodes)
    return st, info


def time_step(st, steps, warmup, use_graph):
    import torch
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        st.run()
        stream.synchronize()
        graph = None
        if use_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                st.run()
        run = graph.replay if graph is not None else st.run
        for _ in range(warmup):
            run()
        stream.synchronize()
    return stream, run


def max_over_ranks(value, device, world):
    """A per-rank duration -> the slowest rank's (what a multi-GPU number is reported as)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed(base, rank):
    """Every rank verifies its own sequence(s): inputs are seeded per rank."""
    return 1000 * base + rank


def time_attention(st, layers, stream, steps, use_graph, sampler=None):
    """The attention launches alone: `layers` launches per repetition, each on its own KV buffers (cold),
    replayed as a graph like the step itself, CUDA events on the launching stream.  At least `steps`
    repetitions, and as many more as it takes to fill MIN_TIMED_SECONDS.  Returns (us per launch, how, reps)."""
    import torch
    with torch.cuda.stream(stream):
        st.seq_len.copy_(st.seq_len0)
        if use_graph:
            graph = torch.cuda.CUDAGraph()
            for layer in range(layers):
                st.verify_attn(layer)
            stream.synchronize()
            with torch.cuda.graph(graph, stream=stream):
                for layer in range(layers):
                    st.verify_attn(layer)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            for _ in range(3):
                graph.replay()
            a1.record(stream)
            stream.synchronize()
            per_replay_s = max(a0.elapsed_time(a1) * 1e-3 / 3, 1e-6)
            reps = max(steps, int(MIN_TIMED_SECONDS / per_replay_s) + 1)
            if sampler is not None:
                sampler.start()
            a0.record(stream)
            for _ in range(reps):
                graph.replay()
            a1.record(stream)
            stream.synchronize()
            # per-replay samples for a median and a minimum beside the mean (50 replays, one event pair each)
            pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(50)]
            for x, y in pairs:
                x.record(stream)
                graph.replay()
                y.record(stream)
            stream.synchronize()
            per = sorted(x.elapsed_time(y) * 1e3 / layers for x, y in pairs)
            time_attention.last_samples = {"median_us_per_launch": per[len(per) // 2], "min_us_per_launch": per[0],
                                           "samples": len(per),
                                           "note": "one event pair per graph replay: includes the replay's launch gap"}
            return (a0.elapsed_time(a1) * 1e3 / (reps * layers),
                    f"CUDA events around {reps} replays of a graph of the {layers} attention launches", reps)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(layers * steps)]
        for rep_i in range(2):                       # first repetition warms up
            if rep_i == 1 and sampler is not None:
                sampler.start()
            i = 0
            for _ in range(steps):
                for layer in range(layers):
                    a, b_ = evs[i]
                    a.record(stream)
                    st.verify_attn(layer)
                    b_.record(stream)
                    i += 1
            stream.synchronize()
        time_attention.last_samples = None
        return (statistics.mean(a.elapsed_time(b_) for a, b_ in evs) * 1e3, "CUDA events around every attention call",
                steps)


time_attention.last_samples = None
# Nominal peaks (context beside the measured ones): HBM3e 8 TB/s, dense bf16 2.25 PFLOP/s.
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}


def attention_roofline(c, info, attn_us, clocks, workload_name, timing, samples=None):
    """The roofline object of the attention kernel for one workload."""
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peaks, peak_src = json.load(open(peaks_path)), "measured"
    else:
        peaks, peak_src = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"
    bytes_alg = attn_algorithmic_bytes(c, info["seq_lens"], info["n_nodes"])
    flops_alg = attn_algorithmic_flops(c, info["seq_lens"], info["depth"])
    t_bytes = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    t_flops = flops_alg / (peaks["bf16_tflops"] * 1e12)
    if t_bytes >= t_flops:
        roof = {"bound": "hbm", "achieved": bytes_alg / (attn_us * 1e-6) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        # a tensor-bound kernel timed in a long region under the power cap (reason flag, or the sampled SM clock well
        # below its maximum) is held against the sustained GEMM figure (seconds-long loop), otherwise against the
        # burst figure; the fraction of the burst figure is reported beside it
        slowed = bool(clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] < 0.9 * clocks["sm_max_mhz"])
        capped = ("sw_power_cap" in (clocks.get("reasons") or []) or slowed) and "bf16_tflops_sustained" in peaks
        achieved = flops_alg / (attn_us * 1e-6) / 1e12
        roof = {"bound": "tensor", "achieved": achieved,
                "peak": peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"], "unit": "TFLOP/s",
                "peak_kind": "sustained (power cap or SM clock below 90 % of its maximum during the timed region)" if capped else "burst",
                "frac_of_burst_peak": achieved / peaks["bf16_tflops"]}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["frac_of_nominal"] = roof["achieved"] / (NOMINAL["hbm_gbs"] if roof["bound"] == "hbm" else NOMINAL["bf16_tflops"])
    samples = samples if samples is not None else time_attention.last_samples
    if samples:
        roof["per_replay"] = samples
    roof["traffic"], roof["traffic_note"] = ncu_traffic(workload_name, bytes_alg)
    roof.update(kernel="tree_attn_kernel", peak_source=peak_src, us_per_launch=attn_us, timing=timing,
                algorithmic_bytes=bytes_alg, algorithmic_flops=flops_alg,
                roofline_us=max(t_bytes, t_flops) * 1e6)
    if clocks.get("sm_mhz"):
        # a latency-bound launch scales with the SM clock: the product lets runs at different clocks be compared
        roof["us_x_sm_mhz"] = attn_us * clocks["sm_mhz"]
    return roof


def sweep_point(name, c, seed, device, steps, sampler_args, layers=None):
    """One more workload for the recorded line: the attention launches alone (no tree construction,
    acceptance or commit timed), on enough layers that the K/V of one repetition is several times the L2."""
    import torch
    from paper_2606_18394_b200.step import VerifyStep
    c = dict(c)
    batch, B, N, W, Hq, Hkv, D = c["batch"], c["B"], c["N"], c["W"], c["Hq"], c["Hkv"], c["D"]
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    rng = np.random.default_rng(seed)
    if c.get("paged"):
        seq = rng.integers(c["L_range"][0], c["L_range"][1] + 1, size=batch).astype(np.int32)
    else:
        seq = np.full(batch, c["L"], dtype=np.int32)
    kv_bytes = int(2 * int(seq.sum()) * Hkv * D * 2)
    layers = layers or max(2, min(c["layers"], int(600e6 // kv_bytes) + 1))
    c["layers"] = layers
    V = 4096                         # the draft vocabulary plays no part in the attention launches
    if c.get("paged"):
        need = [(int(L) + N + 1 + 15) // 16 for L in seq]
        num_pages = sum(need) + 3
        perm = rng.permutation(num_pages)
        table = np.zeros((batch, max(need)), dtype=np.int32)
        pos = 0
        for b, cnt in enumerate(need):
            table[b, :cnt] = perm[pos:pos + cnt]
            pos += cnt
        st = VerifyStep(batch=batch, layers=layers, Hq=Hq, Hkv=Hkv, D=D, B=B, N=N, W=W, V=V,
                        max_seq_len=int(seq.max()), page_size=16, num_pages=num_pages, max_pages=max(need),
                        device=device)
        st.page_table.copy_(torch.from_numpy(table))
    else:
        st = VerifyStep(batch=batch, layers=layers, Hq=Hq, Hkv=Hkv, D=D, B=B, N=N, W=W, V=V,
                        max_seq_len=int(c["L"]), device=device)
    st.seq_len0.copy_(torch.from_numpy(seq))
    for t in (st.q, st.tree_k, st.tree_v):
        t.copy_(torch.randn(t.shape, generator=gen, device=device, dtype=torch.float32))
    for layer in range(layers):
        st.k_cache[layer].copy_(torch.randn(st.k_cache[layer].shape, generator=gen, device=device, dtype=torch.float32))
        st.v_cache[layer].copy_(torch.randn(st.v_cache[layer].shape, generator=gen, device=device, dtype=torch.float32))
    logits = torch.randn(st.logp.shape, generator=gen, device=device, dtype=torch.float32) * 3.0
    top = torch.randint(0, V, (batch, N), generator=gen, device=device)
    logits.scatter_(2, top[:, :, None], 14.0)          # one confident token per depth, so the trees grow deep
    st.logp.copy_(torch.log_softmax(logits.double(), dim=2).float())
    st.root_token.fill_(1)
    st.seq_len.copy_(st.seq_len0)
    st.tree_build()
    torch.cuda.synchronize()
    info = dict(seq_lens=[int(x) for x in seq], depth=st.depth.cpu().numpy(), n_nodes=st.n_nodes.cpu().numpy())
    stream = torch.cuda.Stream()
    sampler = ClockSampler(*sampler_args)
    attn_us, timing, reps = time_attention(st, layers, stream, steps, True, sampler)
    clocks = sampler.stop()
    assert int(st.status.item()) == 0, "a bounded device wait expired"
    roof = attention_roofline(c, info, attn_us, clocks, name, timing)
    point = {"workload": name, "batch": batch, "tree_nodes": B, "prefix": info["seq_lens"] if c.get("paged") else c["L"],
             "layers_timed": layers, "us_per_launch": attn_us, "launches": reps * layers, "clocks": clocks, "roofline": roof}
    del st
    torch.cuda.empty_cache()
    return point


def lm_head_point(c, seed, device, sampler_args, d_model=4096):
    """jet_tree_accept_hidden at the workload's shape: the LM head applied inside the acceptance call, only the
    per-row arg-max kept (no [rows, V] logits in memory).  A weight stream: V * d * 2 bytes from HBM per call;
    several weight copies are cycled so that no call finds its weights in L2."""
    import torch
    import paper_2606_18394_b200 as jet
    batch, B, N, V = c["batch"], c["B"], c["N"], c["V"]
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    rows = batch * B
    hidden = torch.randn((rows, d_model), generator=gen, device=device, dtype=torch.float32).bfloat16()
    copies = 3
    weights = [(torch.randn((V, d_model), generator=gen, device=device, dtype=torch.float32) * 0.02).bfloat16()
               for _ in range(copies)]
    i32 = lambda *shape: torch.zeros(shape, dtype=torch.int32, device=device)
    token, parent, depth = i32(batch, B), i32(batch, B), i32(batch, B)
    parent[:, 0] = -1                                   # a star: every node hangs off the root
    depth[:, 1:] = 1
    anc = i32(batch, B, (B + 31) // 32)
    anc[:, :, 0] = 1
    for v in range(1, B):
        anc[:, v, v // 32] |= (1 << (v % 32)) if v % 32 != 31 else -(1 << 31)
    n_nodes = torch.full((batch,), B, dtype=torch.int32, device=device)
    tgt, acc, path, toks, status = i32(batch, B), i32(batch), i32(batch, N + 1), i32(batch, N + 1), i32(1)
    ws = torch.empty(max(jet.jet_tree_accept_hidden_workspace_bytes(batch, B), 256), dtype=torch.uint8, device=device)

    def call(w):
        jet.jet_tree_accept_hidden(hidden, w, d_model, token, parent, depth, anc, n_nodes, batch, B, V, N, tgt, acc, path,
                                   toks, status, ws)
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        for w in weights:
            call(w)
        stream.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            for w in weights:
                call(w)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(3):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
        reps = max(3, int(MIN_TIMED_SECONDS / max(e0.elapsed_time(e1) * 1e-3 / 3, 1e-6)) + 1)
        sampler = ClockSampler(*sampler_args)
        sampler.start()
        e0.record(stream)
        for _ in range(reps):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
    clocks = sampler.stop()
    assert int(status.item()) == 0, "a bounded device wait expired"
    us = e0.elapsed_time(e1) * 1e3 / (reps * copies)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peaks, src = (json.load(open(peaks_path)), "measured") if os.path.exists(peaks_path) else ({"hbm_gbs": 6650.0}, "fallback")
    bytes_alg = V * d_model * 2 + rows * d_model * 2 + rows * 4
    traffic, note = ncu_traffic("lm_head_accept", bytes_alg)
    roof = {"bound": "hbm", "achieved": bytes_alg / (us * 1e-6) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "kernel": "lm_head_argmax_kernel", "peak_source": src, "us_per_launch": us, "algorithmic_bytes": bytes_alg,
            "algorithmic_flops": 2 * rows * d_model * V, "traffic": traffic, "traffic_note": note,
            "timing": f"CUDA events around {reps} replays of a graph of {copies} calls (memset + GEMM/arg-max + path kernel each)"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    del weights
    torch.cuda.empty_cache()
    return {"workload": "lm_head_accept", "rows": rows, "hidden_size": d_model, "vocab": V, "us_per_call": us,
            "launches": reps * copies * 2, "clocks": clocks, "roofline": roof,
            "note": "replaces jet_tree_accept's scan of fp32 logits when the caller hands over hidden states instead"}


def bench_jet(args):
    import torch
    import torch.distributed as dist
    import paper_2606_18394_b200 as jet

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    jet.load()
    device = f"cuda:{local_rank}"
    torch.cuda.set_device(device)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))
    c = workload(args.config, args.budget, args.batch)
    if args.layers:
        c["layers"] = args.layers
    st, info = build_inputs(c, args.config, rank_seed(2, rank), device, args.score, args.score_alpha, args.layout == "tail",
                            args.draft_input == "logits", args.target_input == "hidden")
    layers = c["layers"]
    if args.accept == "sample":
        assert args.target_input == "logits", "the non-greedy rule needs the target logits"
        st.accept_mode = "sample"
        g = torch.Generator(device=device).manual_seed(rank_seed(3, rank))
        st.u_accept.copy_(torch.rand(st.u_accept.shape, generator=g, device=device))
        st.u_sample.copy_(torch.rand(st.u_sample.shape, generator=g, device=device))

    stream, run = time_step(st, args.steps, max(args.warmup, 3), not args.no_graph)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- device-resident timing of K whole steps
    try:
        gpu_uuid = str(torch.cuda.get_device_properties(device).uuid)
    except Exception:
        gpu_uuid = None
    sampler = ClockSampler(local_rank, gpu_uuid)
    if rank == 0:
        sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(args.steps):
            run()
        e1.record(stream)
    stream.synchronize()
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = max_over_ranks(ms_total, device, world) / args.steps
    # The K steps above may last only a few milliseconds, at whatever clock the GPU happened to run; the same step
    # is timed again over a region of MIN_TIMED_SECONDS with its own clock samples (reported as "sustained").
    sustained = None
    if ms_total * 1e-3 < MIN_TIMED_SECONDS:
        more = int(MIN_TIMED_SECONDS / max(ms_step * 1e-3, 1e-6)) + 1
        sus_sampler = ClockSampler(local_rank, gpu_uuid)
        if rank == 0:
            sus_sampler.start()
        barrier()
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(more):
                run()
            e1.record(stream)
        stream.synchronize()
        barrier()
        sus_ms = max_over_ranks(e0.elapsed_time(e1), device, world) / more
        sus_clocks = sus_sampler.stop() if rank == 0 else None
        if rank == 0:
            sustained = {"steps": more, "ms_per_step": sus_ms, "value": sus_ms * 1e3 / (layers * world), "unit": UNIT,
                         "clocks": sus_clocks}
            if sus_clocks.get("sm_mhz"):
                sustained["value_x_sm_mhz"] = sustained["value"] * sus_clocks["sm_mhz"]
    assert int(st.status.item()) == 0, "a bounded device wait expired"
    acc = st.accept_len.cpu().numpy().tolist()
    if args.accept == "greedy":
        assert acc == info["planted"], (acc, info["planted"])
    else:
        assert all(0 <= a <= c["N"] for a in acc), acc

    # ---------------- the attention launches alone (the dominant kernel), in a region of its own with its own
    #                  clock samples (this is the denominator of roofline.achieved)
    attn_sampler = ClockSampler(local_rank, gpu_uuid)
    attn_us, attn_timing, attn_reps = time_attention(st, layers, stream, args.steps, not args.no_graph,
                                                     attn_sampler if rank == 0 else None)
    attn_clocks = attn_sampler.stop() if rank == 0 else None
    attn_samples = time_attention.last_samples
    assert int(st.status.item()) == 0, "a bounded device wait expired"
    # the same launches issued call by call (no graph): what a caller that does not capture pays per call,
    # host-side argument checks and tensor-map encoding included
    attn_us_eager, _, _ = time_attention(st, layers, stream, max(2, min(args.steps, 10)), False, None)

    # ---------------- end to end: host buffers in, result out, every step
    big = "hidden" if st.accept_mode == "hidden" else "logits"      # the acceptance's input, needed last
    pinned = {k: getattr(st, k).cpu().pin_memory() for k in ("logp", "root_token", big, "q", "tree_k", "tree_v")}
    host_out = {k: torch.empty_like(getattr(st, k), device="cpu").pin_memory()
                for k in ("accept_len", "out_tokens", "path")}
    h2d = sum(v.numel() * v.element_size() for v in pinned.values())
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())

    # The inputs arrive in the order the step needs them, on a copy stream of their own: draft log-probs first, then
    # q / tree K / tree V of the first quarter of the layers, the second ... and last the acceptance's input (the
    # largest, or the hidden states).  The step is cut into graphs at the same places (tree construction, four
    # groups of layers, acceptance + commit); each group starts as soon as its inputs are on the device, so the
    # copies of later layers run under the attention of earlier ones.
    copy_stream = torch.cuda.Stream()
    n_groups = 1 if st.tail else min(4, layers)          # (in-cache tree layout: the tree rows are placed after all copies)
    bounds = [round(i * layers / n_groups) for i in range(n_groups + 1)]
    ev_small, ev_big, back_done = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()
    ev_group = [torch.cuda.Event() for _ in range(n_groups)]

    def part_build():
        st.seq_len.copy_(st.seq_len0)
        st.tree_build()

    def part_group(i):
        for layer in range(bounds[i], bounds[i + 1]):
            st.verify_attn(layer)
    parts = [part_build] + [(lambda i=i: part_group(i)) for i in range(n_groups)] + [st.run_back]
    if not args.no_graph:
        with torch.cuda.stream(stream):
            for f in parts:
                f()
            stream.synchronize()
            graphs = []
            for f in parts:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    f()
                graphs.append(g)
            stream.synchronize()
        parts = [g.replay for g in graphs]
    back_done.record(stream)

    def e2e_step():
        # the copies of this step may start once the step before has finished with the buffers
        copy_stream.wait_event(back_done)
        with torch.cuda.stream(copy_stream):
            for k in ("logp", "root_token"):
                getattr(st, k).copy_(pinned[k], non_blocking=True)
            ev_small.record(copy_stream)
            for i in range(n_groups):
                for k in ("q", "tree_k", "tree_v"):
                    getattr(st, k)[bounds[i]:bounds[i + 1]].copy_(pinned[k][bounds[i]:bounds[i + 1]], non_blocking=True)
                ev_group[i].record(copy_stream)
            getattr(st, big).copy_(pinned[big], non_blocking=True)
            ev_big.record(copy_stream)
        stream.wait_event(ev_small)
        parts[0]()
        for i in range(n_groups):
            stream.wait_event(ev_group[i])
            if st.tail and i == 0:
                st.place_tree()            # the tree's K/V arrive in staging buffers and are put behind the prefixes
            parts[1 + i]()
        stream.wait_event(ev_big)
        parts[-1]()
        back_done.record(stream)
        for k, v in host_out.items():
            v.copy_(getattr(st, k), non_blocking=True)

    with torch.cuda.stream(stream):
        for _ in range(3):
            e2e_step()
        stream.synchronize()
        barrier()
        e0.record(stream)
        for _ in range(args.steps):
            e2e_step()
        e1.record(stream)
        stream.synchronize()
    barrier()
    e2e_ms_step = max_over_ranks(e0.elapsed_time(e1), device, world) / args.steps
    assert host_out["accept_len"].numpy().tolist() == acc

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---------------- roofline of the dominant kernel (one attention call = one tree_attn_kernel launch)
    roof = attention_roofline(c, info, attn_us, attn_clocks, args.config, attn_timing, attn_samples)
    roof["clocks"] = attn_clocks
    roof["us_per_call_without_graph"] = attn_us_eager

    # ---------------- the rest of the metric's range (64 .. 256-node trees at the same layer shape, and the batched
    #                  serving shape): attention launches only, each point timed for MIN_TIMED_SECONDS
    sweep = []
    if args.config == "qwen3_8b" and not args.no_sweep and world == 1:
        base = dict(CONFIGS["qwen3_8b"])
        for nodes in (128, 256):
            cc = dict(base, B=nodes, N=12)
            sweep.append(sweep_point(f"qwen3_8b_b{nodes}", cc, rank_seed(5, rank) + nodes, device, 3,
                                     (local_rank, gpu_uuid)))
        sweep.append(sweep_point("batched_paged", dict(CONFIGS["batched_paged"]), rank_seed(6, rank), device, 3,
                                 (local_rank, gpu_uuid)))
        # the long-generation regime of the same layer shape (prefix 16384): an HBM-bound and a tensor-bound budget
        for nodes in (64, 256):
            cc = dict(CONFIGS["sweep_16k"], B=nodes, N=12 if nodes > 64 else 8)
            sweep.append(sweep_point(f"sweep_16k_b{nodes}", cc, rank_seed(9, rank) + nodes, device, 3,
                                     (local_rank, gpu_uuid)))
        # the draft head's own block-causal attention: a chain of 16 rows (one per draft depth, width 1) over the
        # same context length, at the head's shape; timed over 36 distinct KV buffers so every launch is cold
        sweep.append(sweep_point("draft_head_block16", dict(base, B=16, N=15, W=1), rank_seed(7, rank), device, 3,
                                 (local_rank, gpu_uuid)))
        sweep.append(lm_head_point(c, rank_seed(8, rank), device, (local_rank, gpu_uuid)))

    cpu = cpu_baseline(st, c, info) if not args.no_cpu_baseline else None

    line = {
        "metric": METRIC, "value": ms_step * 1e3 / (layers * world), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.config, "batch_per_gpu": c["batch"], "layers": layers, "Hq": c["Hq"],
                   "Hkv": c["Hkv"], "head_dim": c["D"], "prefix": info["seq_lens"] if c.get("paged") else c["L"],
                   "tree_nodes": c["B"], "max_depth": c["N"], "width": c["W"], "vocab": c["V"],
                   "paged": bool(c.get("paged")), "cuda_graph": not args.no_graph,
                   "layers_overridden": bool(args.layers),
                   "l2": "every layer streams its own KV buffers; one step reads far more than the 126 MB L2",
                   "accepted_len": acc, "accept": args.accept, "tree_kv": args.layout,
                   "score": args.score if args.score != "hybrid" else f"hybrid(alpha={args.score_alpha})",
                   "draft_input": args.draft_input, "target_input": args.target_input},
        "attn_us_per_layer": attn_us,
        "e2e": {"value": e2e_ms_step * 1e3 / (layers * world), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms_step,
                "note": "all inputs come from pinned host memory every step, on a copy stream, in the order the step needs "
                        "them (log-probs, then q / tree K / tree V per quarter of the layers, then the acceptance's input); "
                        "every part of the step starts when its inputs have arrived"},
        "gpu_launches": args.steps * st.launches_per_step(),
        "clocks": clocks, "roofline": roof,
    }
    if sustained is not None:
        line["sustained"] = sustained
    if sweep:
        line["sweep"] = sweep
    if cpu is not None:
        line["cpu_baseline"] = cpu
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
def _bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def oracle_sample(c, x, attn_layers):
    """The CPU oracle on a bounded sample of one step of one sequence: tree_build and tree_accept in
    full, `attn_layers` attention layers in full (fp64).  `x` holds numpy inputs: logp, root, logits,
    planted, scale and per-layer lists q / k / v / tk / tv (bf16 bit patterns).
    Returns (seconds, description, us/layer)."""
    import oracle
    B, N, W, layers = c["B"], c["N"], c["W"], c["layers"]
    t0 = time.perf_counter()
    build = oracle.tree_build_logits_ref if x.get("draft_logits") else oracle.tree_build_ref
    tree = build(x["logp"], x["root"], N, W, B, score_mode=x.get("score_mode", "accum_logp"), alpha=x.get("alpha", 0.0))
    t_build = time.perf_counter() - t0
    t_attn = 0.0
    for layer in range(attn_layers):
        t0 = time.perf_counter()
        oracle.tree_attn_ref(x["q"][layer], x["k"][layer], x["v"][layer], x["tk"][layer], x["tv"][layer],
                             tree["anc_mask"], tree["n_nodes"], x["scale"])
        t_attn += time.perf_counter() - t0
    t0 = time.perf_counter()
    acc = oracle.tree_accept_ref(x["logits"], tree["token"], tree["parent"], tree["depth"], tree["n_nodes"], N)
    t_accept = time.perf_counter() - t0
    per_layer_us = (t_attn / attn_layers + (t_build + t_accept) / layers) * 1e6
    desc = (f"one sequence of the workload: tree_build + tree_accept in full, attention of {attn_layers} of "
            f"{layers} layers in full (fp64); us/layer = attention per layer + (build + accept) / layers; "
            f"commit copies omitted (negligible)")
    if x.get("planted") is not None:
        assert acc["accept_len"] == x["planted"], (acc["accept_len"], x["planted"])
    return t_attn + t_build + t_accept, desc, per_layer_us


def _blas_threads():
    try:
        import threadpoolctl
        info = threadpoolctl.threadpool_info()
        return max(p["num_threads"] for p in info) if info else 1
    except Exception:
        return os.cpu_count()


def cpu_baseline(st, c, info):
    """Oracle timing on the benchmark's own inputs (sequence 0, first two layers), copied to the host."""
    L = info["seq_lens"][0]
    nl = 2
    if st.paged:
        import oracle
        table = st.page_table[0].cpu().numpy()
        ks = [oracle.gather_paged_prefix(_bits(st.k_cache[l]), table, L) for l in range(nl)]
        vs = [oracle.gather_paged_prefix(_bits(st.v_cache[l]), table, L) for l in range(nl)]
    else:
        ks = [_bits(st.k_cache[l, 0, :L]) for l in range(nl)]
        vs = [_bits(st.v_cache[l, 0, :L]) for l in range(nl)]
    if st.accept_mode == "hidden":
        import oracle
        B = st.B
        logits0 = oracle.lm_head_argmax_ref(_bits(st.hidden[:B]), _bits(st.lm_head))["logits"].astype(np.float32)
    else:
        logits0 = st.logits[0].cpu().numpy()
    x = dict(logp=st.logp[0].cpu().numpy(), root=int(st.root_token[0].item()), logits=logits0,
             planted=info["planted"][0], scale=st.scale, q=[_bits(st.q[l, 0]) for l in range(nl)], k=ks, v=vs,
             tk=[_bits(st.tree_k[l, 0]) for l in range(nl)], tv=[_bits(st.tree_v[l, 0]) for l in range(nl)],
             draft_logits=st.draft_logits, score_mode=st.score_mode, alpha=st.score_alpha)
    secs, desc, per_layer_us = oracle_sample(c, x, attn_layers=nl)
    return {"value": per_layer_us, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle", "sample": desc,
            "seconds": secs, "host_cpus": os.cpu_count()}


def reference_inputs(c, seed):
    """Host-only synthetic inputs of the workload's shape for the reference arm (no GPU, no product code)."""
    import oracle
    from jet_inputs import make_attn_inputs, make_logp, make_target_logits
    rng = np.random.default_rng(seed)
    L = c["L"] if "L" in c else int(rng.integers(c["L_range"][0], c["L_range"][1] + 1))
    logp = make_logp(rng, c["N"], c["V"], c["sigma_draft"], peaked_p=0.7)
    tree = oracle.tree_build_ref(logp, 1, c["N"], c["W"], c["B"])
    logits = make_target_logits(rng, c["B"], c["V"], c["sigma_target"])
    _, eff = plant_path(logits, tree["token"], tree["parent"], tree["depth"], tree["n_nodes"], c.get("plant", 4), rng)
    a = make_attn_inputs(rng, c["B"], c["Hq"], c["Hkv"], c["D"], L)
    return dict(logp=logp, root=1, logits=logits, planted=eff, scale=1.0 / np.sqrt(c["D"]), q=[a["q"]],
                k=[a["k_prefix"]], v=[a["v_prefix"]], tk=[a["tree_k"]], tv=[a["tree_v"]])


def bench_reference(args):
    """The reference arm: the CPU oracle as it stands, on the host cores of rank 0 (other ranks idle)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    c = workload(args.config, args.budget, args.batch)
    x = reference_inputs(c, 2000)
    warm = min(args.warmup, 1)
    for _ in range(warm):
        oracle_sample(c, x, attn_layers=1)
    times, per_layer, desc = [], [], ""
    for _ in range(args.steps):
        secs, desc, us = oracle_sample(c, x, attn_layers=1)
        times.append(secs)
        per_layer.append(us)
    value = statistics.mean(per_layer)
    cpu = {"value": value, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle", "sample": desc,
           "host_cpus": os.cpu_count()}
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": warm,
            "ms_per_step": statistics.mean(times) * 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.config, "sample": desc}, "cpu_baseline": cpu,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["jet", "reference"], default="jet")
    ap.add_argument("--config", default="qwen3_8b", choices=list(CONFIGS))
    ap.add_argument("--budget", type=int, default=None, help="tree budget, for the sweep configurations")
    ap.add_argument("--batch", type=int, default=None, help="batch, for configurations that list several")
    ap.add_argument("--layers", type=int, default=None,
                    help="override the workload's layer count (small captures under a profiler; not a bench value)")
    ap.add_argument("--no-graph", action="store_true", help="issue the calls directly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the extra attention-only points of the default run")
    ap.add_argument("--layout", choices=["separate", "tail"], default="separate",
                    help="tree K/V in their own buffers, or in the cache behind each prefix")
    ap.add_argument("--score", choices=["accum_logp", "entropy", "hybrid"], default="accum_logp",
                    help="expansion score of the tree construction (hybrid: --score-alpha)")
    ap.add_argument("--score-alpha", type=float, default=1.0)
    ap.add_argument("--draft-input", choices=["logp", "logits"], default="logp",
                    help="the draft head's output as log-probabilities, or as raw logits (normalised on the fly)")
    ap.add_argument("--target-input", choices=["logits", "hidden"], default="logits",
                    help="what the acceptance is fed with: the target's fp32 logits (the workload as stated), or its final "
                         "hidden states, with the LM head applied inside the call (jet_tree_accept_hidden)")
    ap.add_argument("--accept", choices=["greedy", "sample"], default="greedy",
                    help="acceptance rule of the step: greedy (the headline) or the non-greedy rule at temperature 1")
    args = ap.parse_args()
    if args.impl == "reference":
        bench_reference(args)
    else:
        bench_jet(args)


if __name__ == "__main__":
    main()
