#!/usr/bin/env python
"""Benchmark of the draft-and-verify hot path: microseconds per draft-tree cycle.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama3_8b] [--impl ours|reference]

A step is one whole cycle (D x expand, rerank, tree mask, one tree attention per layer, accept, KV
compaction) on seeded synthetic inputs that are resident in HBM, replayed as one CUDA graph.  Rank 0
prints one JSON line.  With N > 1 every rank runs an independent replica (the path has no exchange
step); the value is then the time per cycle over all replicas.

``--impl reference`` times the CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import generators as gen  # noqa: E402
from workloads import get_config  # noqa: E402

METRIC = "us_per_draft_tree_cycle"
N_SETS = 4  # rotating logit sets: 4 x (draft + target rows) is larger than the 126 MB L2

# DRAM bytes of one tree-attention call (attention kernel 17,596,030 + merge kernel 4,618,880; the
# merge's are the partial rows that ncu's cache flush between captured launches pushed out of L2), from
# the ncu capture summarised under profiles/ (None: not captured for that workload)
NCU_DRAM_BYTES_PER_LAUNCH = {"llama3_8b": 17596030 + 4618880}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops_sustained", 1400.0)), "measured"
    return 6650.0, 1400.0, "fallback"


# ------------------------------------------------------------------------------------------------
# clocks during the timed region

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed work runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.02)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)

def oracle_cycle_seconds(cfg, seed: int = 0, attn_samples: int = 96, threads: int | None = None):
    """Times the oracle on a bounded sample of one cycle and extrapolates to the whole cycle.
    Logit steps and tree steps run whole; attention runs `attn_samples` query rows of one layer and is
    scaled to n_layers * m * Hq rows; compaction runs on one layer and is scaled to n_layers.
    `threads`: run the oracle's loops over independent units on that many threads (default: all)."""
    from oracle import ref
    if threads is not None:
        before = ref.set_threads(threads)
        try:
            return oracle_cycle_seconds(cfg, seed, attn_samples)
        finally:
            ref.set_threads(before)
    small = cfg.with_(B=1)
    t = {}
    draft = gen.draft_rows(small, seed)
    t0 = time.perf_counter()
    tree = ref.build_tree(draft, small.V, small.k, small.D)
    t["expand"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    sel = ref.rerank(tree.token, tree.parent, tree.value, small.k, small.D, small.m)
    kv_len = gen.kv_lengths(small, seed)
    bits, _, _, _ = ref.tree_mask(sel.parent, sel.depth, sel.n_sel, kv_len, small.m)
    t["rerank_mask"] = time.perf_counter() - t0
    kv_off = gen.kv_offsets(kv_len, small.m)
    q, kc, vc = gen.qkv_bf16(small, seed, kv_len, kv_off)
    rng = np.random.default_rng(seed)
    samples = np.stack([np.zeros(attn_samples, np.int64), rng.integers(0, small.Hq, attn_samples),
                        rng.integers(0, small.m, attn_samples)], axis=1).astype(np.int32)
    t0 = time.perf_counter()
    ref.tree_attention(q, kc, vc, kv_off, kv_len, bits, 1.0 / math.sqrt(small.d), samples=samples)
    per_row = (time.perf_counter() - t0) / attn_samples
    t["attention_extrapolated"] = per_row * small.m * small.Hq * small.n_layers
    target = gen.target_rows(small, seed, draft, tree.parent, sel.index)
    ua, ub = gen.uniforms(small, seed)
    t0 = time.perf_counter()
    acc = ref.accept(target, draft if small.temperature > 0 else None, sel, small.V, small.k, small.D,
                     small.m, small.temperature, ua, ub)
    t["accept"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    ref.kv_compact([kc], [vc], kv_off, kv_len.copy(), acc.acc_path, acc.acc_len, small.m, small.D)
    t["kv_compact_extrapolated"] = (time.perf_counter() - t0) * small.n_layers
    total = sum(t.values())
    sample = (f"B=1 of {cfg.name}: expand/rerank/mask/accept whole; attention {attn_samples} of "
              f"{small.m * small.Hq * small.n_layers} query rows (1 layer) scaled; compaction 1 of "
              f"{small.n_layers} layers scaled")
    return total, t, sample, ref.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = get_config(args.workload)
    steps, warmup = max(1, min(args.steps, 3)), min(args.warmup, 1)
    for _ in range(warmup):
        oracle_cycle_seconds(cfg, attn_samples=32)
    t0 = time.perf_counter()
    last = None
    for _ in range(steps):
        last = oracle_cycle_seconds(cfg)
    wall = (time.perf_counter() - t0) / steps
    total, parts, sample, cores = last
    us = total * 1e6
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": wall * 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "B": 1, "note": "oracle cycle time extrapolated from a bounded sample"},
        "cpu_baseline": {"value": us, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample,
                         "parts_us": {k: v * 1e6 for k, v in parts.items()}},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def max_over_ranks(value: float, world: int, device=None) -> float:
    """The slowest rank's time: a single-element all-reduce (MAX) over the default process group."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_seed(rank: int) -> int:
    """Every replica draws its own inputs."""
    return 1000 * rank


def batched_attention_extra(e2, dev, stream, hbm_peak, B=32, n_layers=3, reps=10):
    """Tree attention alone at the batched, ragged LLaMA3-8B-shaped workload: the regime in which a
    launch moves enough bytes (about 0.6 GB per layer) for the HBM fraction to be about the kernel
    rather than about launch latency.  Attention-only, a few distinct layers larger than L2."""
    import torch
    cfg = get_config("llama3_8b_batched").with_(B=B)
    kv_len_h = gen.kv_lengths(cfg, 0)
    kv_off_h = gen.kv_offsets(kv_len_h, cfg.m)
    rows = int(kv_off_h[-1] + kv_len_h[-1] + cfg.m)
    max_len = int(kv_len_h.max())
    g = torch.Generator(device=dev).manual_seed(99)
    ks = [torch.randn((rows, cfg.Hkv, cfg.d), generator=g, device=dev).to(torch.bfloat16) for _ in range(n_layers)]
    vs = [torch.randn((rows, cfg.Hkv, cfg.d), generator=g, device=dev).to(torch.bfloat16) for _ in range(n_layers)]
    q = torch.randn((B, cfg.m, cfg.Hq, cfg.d), generator=g, device=dev).to(torch.bfloat16)
    out = torch.zeros_like(q)
    W = (cfg.m + 63) // 64
    mask = torch.zeros((B, cfg.m, W), dtype=torch.int64, device=dev)
    for i in range(cfg.m):  # a chain: token i sees tokens 0..i
        mask[:, i, 0] = (1 << (i + 1)) - 1
    kv_off, kv_len = torch.from_numpy(kv_off_h).to(dev), torch.from_numpy(kv_len_h).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(max(e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=B, m=cfg.m, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d,
                                            max_kv_len=max_len), 256), dtype=torch.uint8, device=dev)
    e2.workspace_init(ws)
    torch.cuda.synchronize()  # inputs were made on the default stream; the timed work runs on `stream`

    def layers():
        for kc, vc in zip(ks, vs):
            e2.tree_attention(q, kc, vc, rows, kv_off, kv_len, mask, B, cfg.m, cfg.Hq, cfg.Hkv, cfg.d, max_len,
                              1.0 / math.sqrt(cfg.d), out, None, ws, status)

    with torch.cuda.stream(stream):
        for _ in range(3):
            layers()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(reps):
            layers()
        ev1.record(stream)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    us = ev0.elapsed_time(ev1) * 1e3 / (reps * n_layers)
    nbytes = float(sum(2 * (int(L) + cfg.m) * cfg.Hkv * cfg.d * 2 for L in kv_len_h)) + 2.0 * B * cfg.m * cfg.Hq * cfg.d * 2
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"workload": f"llama3_8b_batched B={B}, ragged kv_len {int(kv_len_h.min())}..{max_len}",
            "us_per_layer": us, "algorithmic_bytes_per_layer": nbytes, "achieved_gbs": gbs, "frac_of_measured_hbm": gbs / hbm_peak}


def batched_expand_extra(e2, dev, stream, hbm_peak, B=128, n_sets=None, reps=20):
    """One expansion step (k rows per sequence) alone at a batch that gives a launch enough bytes
    (B*k*V*4 = 0.66 GB) for the HBM fraction to be about the kernel; a few distinct logit sets
    larger than L2."""
    import torch
    cfg = get_config("llama3_8b").with_(B=B)
    k, V, D = cfg.k, cfg.V, cfg.D
    if n_sets is None:
        n_sets = int(max(4, math.ceil(300e6 / (B * k * V * 4.0))))
    reps = max(2, min(reps, 400 // n_sets))
    g = torch.Generator(device=dev).manual_seed(7)
    logits = [torch.randn((B, k, V), generator=g, device=dev) for _ in range(n_sets)]
    N = k + (D - 1) * k * k
    token = torch.zeros((B, N), dtype=torch.int32, device=dev)
    parent = torch.zeros_like(token)
    value = torch.zeros((B, N), dtype=torch.float64, device=dev)
    frontier0 = torch.arange(k, dtype=torch.int32, device=dev).repeat(B, 1).contiguous()  # the step-0 nodes
    frontier = frontier0.clone()
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(e2.workspace_bytes(e2.OP_EXPAND, B=B, V=V, k=k, D=D), dtype=torch.uint8, device=dev)
    e2.workspace_init(ws)
    torch.cuda.synchronize()  # inputs were made on the default stream; the timed work runs on `stream`

    def steps():
        for z in logits:
            frontier.copy_(frontier0)  # every call expands the same level
            e2.expand(z, k * V, B, V, k, D, 1, token, parent, value, frontier, ws, status)

    with torch.cuda.stream(stream):
        for _ in range(3):
            steps()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(reps):
            steps()
        ev1.record(stream)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, f"device status {int(status.item())} in the expansion sweep at B={B}"
    us = ev0.elapsed_time(ev1) * 1e3 / (reps * n_sets)  # includes the 5 KB frontier reset per call
    nbytes = float(B) * k * V * 4
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"workload": f"llama3_8b expansion step 1, B={B} ({B * k} rows of {V} logits)", "us_per_call": us,
            "algorithmic_bytes_per_call": nbytes, "achieved_gbs": gbs, "frac_of_measured_hbm": gbs / hbm_peak}


def batched_accept_extra(e2, dev, stream, hbm_peak, B=16, reps=10):
    """Acceptance at temperature 1 alone for B sequences of the LLaMA3-8B-shaped tree: per sequence the
    target and draft rows of every node that has selected children are read (once each), plus the
    two rows of the stopping node for the extra token.  One input set (0.9 GB) is larger than L2."""
    import torch
    from paper_2406_16858_b200.cycle import CycleBuffers, CycleShape
    cfg = get_config("llama3_8b").with_(B=B, temperature=1.0)
    shape = CycleShape(cfg.B, cfg.V, cfg.k, cfg.D, cfg.m, 1, cfg.Hq, cfg.Hkv, cfg.d, 64, cfg.temperature)
    buf = CycleBuffers(shape, dev)
    g = torch.Generator(device=dev).manual_seed(11)
    draft = torch.from_numpy(gen.draft_rows(cfg, 5)).to(dev)
    kv_len = torch.zeros(B, dtype=torch.int32, device=dev)
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        buf.expand_all(draft)
        buf.rerank_and_mask(kv_len)
    torch.cuda.synchronize()
    nd = gen.node_draft_rows(buf.tree_parent.cpu().numpy(), cfg.k, cfg.D)
    sel_index, sel_parent = buf.sel_index.cpu().numpy(), buf.sel_parent.cpu().numpy()
    src_rows = np.zeros((B, cfg.m + 1), np.int64)
    parents = 0  # nodes (the root included) with at least one selected child
    for b in range(B):
        for x in range(cfg.m):
            r = nd[b, sel_index[b, x]] if sel_index[b, x] >= 0 else -1
            src_rows[b, 1 + x] = r if r >= 0 else (x * 7 + 3) % cfg.R
        parents += len(set(int(q) for q, i in zip(sel_parent[b], sel_index[b]) if i >= 0))
    base = torch.gather(draft, 1, torch.from_numpy(src_rows).to(dev)[:, :, None].expand(-1, -1, cfg.V))
    target = (base + 0.5 * torch.randn(base.shape, generator=g, device=dev)).contiguous()
    del base
    ua_h, ub_h = gen.uniforms(cfg, 5)
    ua, ub = torch.from_numpy(ua_h).to(dev), torch.from_numpy(ub_h).to(dev)
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for _ in range(3):
            buf.accept(target, draft, ua, ub)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(reps):
            buf.accept(target, draft, ua, ub)
        ev1.record(stream)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    us = ev0.elapsed_time(ev1) * 1e3 / reps
    nbytes = float(parents + B) * 2 * cfg.V * 4
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"workload": f"llama3_8b acceptance at temperature 1, B={B} ({parents} nodes with selected children)",
            "us_per_call": us, "algorithmic_bytes_per_call": nbytes, "achieved_gbs": gbs,
            "frac_of_measured_hbm": gbs / hbm_peak}


def draft_attention_extra(e2, dev, stream, hbm_peak, reps=200):
    """The draft model's own attention during expansion (one decoder layer with the target's head
    geometry): at step s its s*k tokens fed so far are the tree rows, the k newest are the step's
    queries.  Same entry point as the verification pass, m = s*k; a chain-shaped mask stands in for
    the tree's; 8 rotating caches (136 MB) are larger than L2."""
    import torch
    cfg = get_config("llama3_8b")
    L, k, D = int(cfg.kv_len), cfg.k, cfg.D
    g = torch.Generator(device=dev).manual_seed(3)
    m_max = (D - 1) * k
    rows = L + m_max
    n_sets = 8
    ks = [torch.randn((rows, cfg.Hkv, cfg.d), generator=g, device=dev).to(torch.bfloat16) for _ in range(n_sets)]
    vs = [torch.randn((rows, cfg.Hkv, cfg.d), generator=g, device=dev).to(torch.bfloat16) for _ in range(n_sets)]
    kv_off = torch.zeros(1, dtype=torch.int64, device=dev)
    kv_len = torch.full((1,), L, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    scale = 1.0 / math.sqrt(cfg.d)
    per_step = []
    for s in range(1, D):
        m = s * k
        q = torch.randn((1, m, cfg.Hq, cfg.d), generator=g, device=dev).to(torch.bfloat16)
        out = torch.zeros_like(q)
        mask = torch.zeros((1, m, 1), dtype=torch.int64, device=dev)
        for i in range(m):  # token i sees itself and the tokens k, 2k, ... before it
            bits = 0
            j = i
            while j >= 0:
                bits |= 1 << j
                j -= k
            mask[0, i, 0] = bits
        ws = torch.empty(max(e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=1, m=m, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d,
                                                max_kv_len=L), 256), dtype=torch.uint8, device=dev)
        e2.workspace_init(ws)
        torch.cuda.synchronize()  # inputs were made on the default stream; the timed work runs on `stream`

        def calls():
            for kc, vc in zip(ks, vs):
                e2.tree_attention(q, kc, vc, rows, kv_off, kv_len, mask, 1, m, cfg.Hq, cfg.Hkv, cfg.d, L, scale, out,
                                  None, ws, status)

        with torch.cuda.stream(stream):
            calls()
            stream.synchronize()
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=stream):
                calls()
            for _ in range(3):
                gr.replay()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            for _ in range(reps // n_sets):
                gr.replay()
            ev1.record(stream)
        torch.cuda.synchronize()
        per_step.append(ev0.elapsed_time(ev1) * 1e3 / ((reps // n_sets) * n_sets))
    assert int(status.item()) == 0
    nbytes = 2.0 * (L + m_max) * cfg.Hkv * cfg.d * 2
    return {"workload": f"llama3_8b-shaped draft layer, kv_len {L}, steps 1..{D - 1} with m = {k}..{m_max}",
            "us_per_step": per_step, "us_all_steps": float(sum(per_step)),
            "frac_of_measured_hbm_last_step": nbytes / (per_step[-1] * 1e-6) / 1e9 / hbm_peak}


# ------------------------------------------------------------------------------------------------
# the CUDA path

def lm_head_extra(e2, dev, stream, hbm_peak, reps=30):
    """The LM head in front of each expansion step (Section 4.1) at the llama3_8b shape: k feature rows
    of hidden size 4096 against a random bf16 [V][4096] weight matrix (1.05 GB, larger than L2), alone
    and followed by the expansion that ranks its logits.  Algorithmic bytes per launch: the weight
    matrix once, plus features and logits."""
    import torch
    cfg = get_config("llama3_8b")
    H, V, k, D = 4096, cfg.V, cfg.k, cfg.D
    g = torch.Generator(device=dev).manual_seed(5)
    weight = (torch.randn((V, H), generator=g, device=dev) * (2.0 / math.sqrt(H))).to(torch.bfloat16)
    hidden = torch.randn((k, H), generator=g, device=dev).to(torch.bfloat16)
    logits = torch.zeros((k, V), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    N = k + (D - 1) * k * k
    token = torch.zeros((1, N), dtype=torch.int32, device=dev)
    parent = torch.zeros((1, N), dtype=torch.int32, device=dev)
    value = torch.zeros((1, N), dtype=torch.float64, device=dev)
    frontier = torch.zeros((1, k), dtype=torch.int32, device=dev)
    ws = torch.empty(max(e2.workspace_bytes(e2.OP_EXPAND, B=1, V=V, k=k, D=D), 256), dtype=torch.uint8, device=dev)
    e2.workspace_init(ws)
    torch.cuda.synchronize()  # inputs were made on the default stream; the timed work runs on `stream`
    out = {}
    for name in ("lm_head", "lm_head_then_expand"):
        def calls():
            e2.lm_head(hidden, weight, k, H, V, logits, status)
            if name == "lm_head_then_expand":  # level 1 again from the first row, then level 2 from all k rows
                e2.expand(logits, k * V, 1, V, k, D, 0, token, parent, value, frontier, ws, status)
                e2.expand(logits, k * V, 1, V, k, D, 1, token, parent, value, frontier, ws, status)
        with torch.cuda.stream(stream):
            for _ in range(3):
                calls()
            stream.synchronize()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            for _ in range(reps):
                calls()
            ev1.record(stream)
        torch.cuda.synchronize()
        out[name + "_us"] = ev0.elapsed_time(ev1) * 1e3 / reps
    assert int(status.item()) == 0
    nbytes = 2.0 * V * H + 2.0 * k * H + 4.0 * k * V
    out.update({"workload": f"llama3_8b-shaped LM head, {k} rows x {H} -> {V} logits, "
                            f"bf16 weights {2.0 * V * H / 1e9:.2f} GB",
                "bytes_per_launch": nbytes, "achieved_gbs": nbytes / (out["lm_head_us"] * 1e-6) / 1e9,
                "frac_of_measured_hbm": nbytes / (out["lm_head_us"] * 1e-6) / 1e9 / hbm_peak})
    return out


def lm_head_fused_extra(e2, dev, stream, hbm_peak, reps=10):
    """The LM head in front of a batched expansion step at the llama3_8b shape, 16 and 32 sequences
    (160 and 320 feature rows): the two chained calls (logits written, then ranked) against the fused
    call that never writes them.  Algorithmic bytes of the fused step: the weight matrix once per
    256 rows."""
    import torch
    cfg = get_config("llama3_8b")
    H, V, k, D = 4096, cfg.V, cfg.k, cfg.D
    g = torch.Generator(device=dev).manual_seed(6)
    weight = (torch.randn((V, H), generator=g, device=dev) * (2.0 / math.sqrt(H))).to(torch.bfloat16)
    out = []
    for B in (16, 32):
        rows = B * k
        hidden = torch.randn((rows, H), generator=g, device=dev).to(torch.bfloat16)
        logits = torch.zeros((rows, V), dtype=torch.float32, device=dev)
        N = k + (D - 1) * k * k
        token = torch.zeros((B, N), dtype=torch.int32, device=dev)
        parent = torch.zeros((B, N), dtype=torch.int32, device=dev)
        value = torch.zeros((B, N), dtype=torch.float64, device=dev)
        frontier0 = torch.arange(k, dtype=torch.int32, device=dev).repeat(B, 1).contiguous()
        frontier = frontier0.clone()
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        ws = torch.empty(max(e2.workspace_bytes(e2.OP_EXPAND, B=B, V=V, k=k, D=D),
                             e2.workspace_bytes(e2.OP_LM_HEAD_EXPAND, B=B, V=V, k=k, D=D), 256), dtype=torch.uint8, device=dev)
        e2.workspace_init(ws)
        torch.cuda.synchronize()
        res = {"B": B, "rows": rows}
        for name in ("chained", "fused"):
            def calls():
                frontier.copy_(frontier0)  # every call expands the same level
                if name == "chained":
                    e2.lm_head(hidden, weight, rows, H, V, logits, status)
                    e2.expand(logits, k * V, B, V, k, D, 1, token, parent, value, frontier, ws, status)
                else:
                    e2.lm_head_expand(hidden, weight, H, B, V, k, D, 1, token, parent, value, frontier, ws, status)
            with torch.cuda.stream(stream):
                for _ in range(2):
                    calls()
                stream.synchronize()
                ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                ev0.record(stream)
                for _ in range(reps):
                    calls()
                ev1.record(stream)
            torch.cuda.synchronize()
            res[name + "_us"] = ev0.elapsed_time(ev1) * 1e3 / reps
        assert int(status.item()) == 0
        passes = (rows + 255) // 256
        nbytes = 2.0 * V * H * passes + 2.0 * rows * H
        res.update({"fused_algorithmic_bytes": nbytes, "fused_achieved_gbs": nbytes / (res["fused_us"] * 1e-6) / 1e9,
                    "fused_frac_of_measured_hbm": nbytes / (res["fused_us"] * 1e-6) / 1e9 / hbm_peak,
                    "chained_logit_bytes_written_and_read": 8.0 * rows * V,
                    "fused_tflops": 2.0 * rows * V * H / (res["fused_us"] * 1e-6) / 1e12})
        out.append(res)
        del hidden, logits, ws
    return {"workload": f"llama3_8b-shaped LM head ({H} -> {V}) + expansion step 1, bf16 weights {2.0 * V * H / 1e9:.2f} GB", "cases": out}


def side_measurements(e2, dev, stream, hbm_peak, only=""):
    """The measurements beside the bench line, by key; `only`: comma-separated keys (default: all)."""
    table = {
        "attention_batched": lambda: batched_attention_extra(e2, dev, stream, hbm_peak),
        "expand_batched": lambda: batched_expand_extra(e2, dev, stream, hbm_peak),
        "expand_sweep": lambda: [dict(B=b, **{k_: v for k_, v in batched_expand_extra(e2, dev, stream, hbm_peak, B=b).items()
                                              if k_ != "workload"}) for b in (1, 8, 32)],
        "accept_batched": lambda: batched_accept_extra(e2, dev, stream, hbm_peak),
        "accept_batched_b32": lambda: batched_accept_extra(e2, dev, stream, hbm_peak, B=32),
        "draft_attention": lambda: draft_attention_extra(e2, dev, stream, hbm_peak),
        "lm_head": lambda: lm_head_extra(e2, dev, stream, hbm_peak),
        "lm_head_fused": lambda: lm_head_fused_extra(e2, dev, stream, hbm_peak),
    }
    want = [w for w in only.split(",") if w] or list(table)
    unknown = [w for w in want if w not in table]
    if unknown:
        raise SystemExit(f"unknown side measurement(s) {unknown}; known: {sorted(table)}")
    return {w: table[w]() for w in want}


def run_ours(args):
    import torch

    import paper_2406_16858_b200 as e2
    from paper_2406_16858_b200.cycle import CycleBuffers, CycleShape, enqueue_cycle

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    if args.extras_only:  # side measurements alone (one GPU; also what the ncu summaries capture)
        stream = torch.cuda.Stream(device=dev)
        print(json.dumps(side_measurements(e2, dev, stream, _peaks()[0], args.extras)))
        return
    cfg = get_config(args.workload)
    if args.batch:
        cfg = cfg.with_(B=args.batch)
    if args.temperature is not None:
        cfg = cfg.with_(temperature=args.temperature)
    seed = replica_seed(rank)
    kv_len_h = gen.kv_lengths(cfg, seed)
    kv_off_h = gen.kv_offsets(kv_len_h, cfg.m)
    rows = int(kv_off_h[-1] + kv_len_h[-1] + cfg.m)
    max_len = int(kv_len_h.max())
    shape = CycleShape(cfg.B, cfg.V, cfg.k, cfg.D, cfg.m, cfg.n_layers, cfg.Hq, cfg.Hkv, cfg.d, max_len,
                       cfg.temperature)
    scale = 1.0 / math.sqrt(cfg.d)
    g = torch.Generator(device=dev).manual_seed(seed + 1)

    # ---- inputs resident in HBM ------------------------------------------------------------------
    def randn_bf16(*shape_):
        return torch.randn(shape_, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)

    # One allocation each for all layers' K, V, Q and O, handed to the library layer by layer: the end
    # to end region below then moves a cycle's per-layer inputs and results in a handful of copies.
    k_all = torch.empty((cfg.n_layers, rows, cfg.Hkv, cfg.d), dtype=torch.bfloat16, device=dev)
    v_all = torch.empty_like(k_all)
    for layer in range(cfg.n_layers):
        k_all[layer].copy_(randn_bf16(rows, cfg.Hkv, cfg.d))
        v_all[layer].copy_(randn_bf16(rows, cfg.Hkv, cfg.d))
    q_all = randn_bf16(cfg.n_layers, cfg.B, cfg.m, cfg.Hq, cfg.d)
    out_all = torch.zeros_like(q_all)
    k_layers, v_layers = list(k_all.unbind(0)), list(v_all.unbind(0))
    q_layers, out_layers = list(q_all.unbind(0)), list(out_all.unbind(0))
    k_ptrs = torch.tensor([t.data_ptr() for t in k_layers], dtype=torch.int64, device=dev)
    v_ptrs = torch.tensor([t.data_ptr() for t in v_layers], dtype=torch.int64, device=dev)
    kv_off = torch.from_numpy(kv_off_h).to(dev)
    kv_len0 = torch.from_numpy(kv_len_h).to(dev)
    kv_len = kv_len0.clone()

    # one set of tree/selection arrays per logit set (a set's acceptance reads its own tree's selection);
    # the scratch workspace is shared
    bufs = [CycleBuffers(shape, dev) for _ in range(N_SETS)]
    for bb in bufs[1:]:
        bb.ws = bufs[0].ws
    sets = []
    for i in range(N_SETS):
        buf = bufs[i]
        draft_h = gen.draft_rows(cfg, seed + 17 * i)
        draft = torch.from_numpy(draft_h).to(dev)
        # the target rows depend on which nodes were selected: build the tree once to find them
        buf.expand_all(draft)
        buf.rerank_and_mask(kv_len)
        torch.cuda.synchronize()
        nd = gen.node_draft_rows(buf.tree_parent.cpu().numpy(), cfg.k, cfg.D)
        sel_index = buf.sel_index.cpu().numpy()
        src_rows = np.zeros((cfg.B, cfg.m + 1), np.int64)
        for b in range(cfg.B):
            for x in range(cfg.m):
                r = nd[b, sel_index[b, x]] if sel_index[b, x] >= 0 else -1
                src_rows[b, 1 + x] = r if r >= 0 else (x * 7 + 3) % cfg.R  # stand-in row for unexpanded nodes
        base = torch.gather(draft, 1, torch.from_numpy(src_rows).to(dev)[:, :, None].expand(-1, -1, cfg.V))
        target = base + 0.5 * torch.randn(base.shape, generator=g, device=dev)
        ua_h, ub_h = gen.uniforms(cfg, seed + 17 * i)
        sets.append(dict(buf=buf, draft=draft, target=target.contiguous(), ua=torch.from_numpy(ua_h).to(dev),
                         ub=torch.from_numpy(ub_h).to(dev)))
    assert all(int(bb.status.item()) == 0 for bb in bufs), "device status raised while preparing inputs"
    buf = bufs[0]
    # The sets read the same queries and write the same outputs, but the second set has copies of its
    # own: the end to end region uploads a step's queries while the cycle of the step before (the other
    # set) still reads its own, and reads a step's outputs back while the next cycle writes the other's.
    q_alt, out_alt = q_all.clone(), torch.zeros_like(out_all)
    for i, s in enumerate(sets):
        s["q_all"] = q_alt if i == 1 else q_all
        s["q_layers"] = list(s["q_all"].unbind(0))
        s["out_all"] = out_alt if i == 1 else out_all
        s["out_layers"] = list(s["out_all"].unbind(0))

    def one_cycle(s):
        kv_len.copy_(kv_len0)  # the cache length is caller state: start every cycle from the same prefix
        enqueue_cycle(s["buf"], s["draft"], s["target"], s["ua"], s["ub"], s["q_layers"], k_layers, v_layers,
                      s["out_layers"], k_ptrs, v_ptrs, kv_off, kv_len, scale)

    stream = torch.cuda.Stream(device=dev)
    graphs = []
    with torch.cuda.stream(stream):
        one_cycle(sets[0])  # warm every kernel (lazy module load) before capture
        stream.synchronize()
        for s in sets:
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=stream):
                one_cycle(s)
            graphs.append(gr)
        # attention alone (all layers) for the roofline of the dominant kernel
        attn_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(attn_graph, stream=stream):
            for qq, kc, vc, oo in zip(q_layers, k_layers, v_layers, out_layers):
                buf.attention(qq, kc, vc, kv_off, kv_len0, oo, scale)
        # the other steps on their own, for the per-step breakdown
        step_graphs = {}  # one graph per logit set and step, replayed in rotation: the logits come from HBM
        for name, fn in (("expand_x%d" % cfg.D, lambda z: z["buf"].expand_all(z["draft"])),
                         ("rerank_mask", lambda z: z["buf"].rerank_and_mask(kv_len0)),
                         ("accept", lambda z: z["buf"].accept(z["target"], z["draft"], z["ua"], z["ub"]))):
            step_graphs[name] = []
            for z in sets:
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=stream):
                    fn(z)
                step_graphs[name].append(gr)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with torch.cuda.stream(stream):
            ev0.record(stream)
            for i in range(steps):
                fn(i)
            ev1.record(stream)
        barrier()
        return max_over_ranks(ev0.elapsed_time(ev1), world, dev)

    def timed_each(fn, steps):
        """Per-step device times (ms): an event between consecutive steps."""
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        barrier()
        with torch.cuda.stream(stream):
            evs[0].record(stream)
            for i in range(steps):
                fn(i)
                evs[i + 1].record(stream)
        barrier()
        return [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]

    def spread(ms_list, per=1.0):
        a = np.asarray(ms_list) * 1e3 / per
        return {"median": float(np.median(a)), "p10": float(np.percentile(a, 10)), "p90": float(np.percentile(a, 90)),
                "n": int(a.size)}

    kv_bytes = float(sum(2 * (int(L) + cfg.m) * cfg.Hkv * cfg.d * 2 for L in kv_len_h))
    qo_bytes = float(2 * cfg.B * cfg.m * cfg.Hq * cfg.d * 2)
    attn_bytes = kv_bytes + qo_bytes  # algorithmic bytes of one tree-attention call (one layer)

    K, W = args.steps, max(args.warmup, 3)
    with ClockSampler(local) as clocks:
        timed(lambda i: graphs[i % N_SETS].replay(), W)
        ms_total = timed(lambda i: graphs[i % N_SETS].replay(), K)
        cycle_spread = spread(timed_each(lambda i: graphs[i % N_SETS].replay(), max(20, min(K, 200))))
        attn_reps = max(20, min(K, 400))
        timed(lambda i: attn_graph.replay(), 3)
        ms_attn = timed(lambda i: attn_graph.replay(), attn_reps)
        attn_spread = spread(timed_each(lambda i: attn_graph.replay(), min(attn_reps, 100)), per=cfg.n_layers)
        breakdown = {"tree_attention_x%d" % cfg.n_layers: ms_attn * 1e3 / attn_reps}
        breakdown_spread = {}
        for name, grs in step_graphs.items():
            timed(lambda i: grs[i % N_SETS].replay(), 4)
            breakdown[name] = timed(lambda i: grs[i % N_SETS].replay(), 48) * 1e3 / 48
            breakdown_spread[name] = spread(timed_each(lambda i: grs[i % N_SETS].replay(), 48))
        # launch-granularity floor: what a stream of plain device-to-device copies of the same sizes
        # costs per launch when replayed as a graph (one layer's K/V + Q/O bytes; one expansion call's logits)
        floor = {}
        for name, nbytes in (("attention_layer", int(attn_bytes)), ("expand_call", cfg.B * cfg.k * cfg.V * 4)):
            n_src = int(min(32, max(2, math.ceil(400e6 / nbytes))))  # together larger than L2
            src = [torch.empty(nbytes, dtype=torch.uint8, device=dev).random_(0, 255) for _ in range(n_src)]
            dst = torch.empty(nbytes, dtype=torch.uint8, device=dev)
            with torch.cuda.stream(stream):
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=stream):
                    for t in src:
                        dst.copy_(t)
            timed(lambda i: gr.replay(), 3)
            us = timed(lambda i: gr.replay(), 20) * 1e3 / (20 * n_src)
            floor[name] = {"bytes_per_launch": nbytes, "us_per_launch": us, "read_gbs": nbytes / (us * 1e-6) / 1e9,
                           "note": f"graph of {n_src} cudaMemcpyAsync device-to-device, distinct sources (larger than L2 together), one destination"}
            del src, dst, gr

        # ---- end to end: inputs start in pinned host memory, results end in host memory -------------
        host_in = {
            "draft": sets[0]["draft"].cpu().pin_memory(), "target": sets[0]["target"].cpu().pin_memory(),
            "ua": sets[0]["ua"].cpu().pin_memory(), "ub": sets[0]["ub"].cpu().pin_memory(),
            "q": q_all.cpu().pin_memory(),
        }
        # the K/V of the m tree tokens are this cycle's new cache rows, one block per layer
        tree_rows = [(b, int(kv_off_h[b] + kv_len_h[b])) for b in range(cfg.B)]
        # [layer][K or V][sequence][m][Hkv][d]: one upload into a staging tensor, then one strided
        # device copy per sequence and operand puts the rows behind the sequence's prefix in every layer
        host_in["tree_kv"] = torch.stack([torch.stack([c[:, r:r + cfg.m] for _, r in tree_rows], dim=1)
                                          for c in (k_all, v_all)], dim=1).cpu().pin_memory()
        tree_kv_dev = [torch.empty_like(host_in["tree_kv"], device=dev) for _ in range(2)]  # one per alternating set
        host_out = {"acc_len": torch.zeros(cfg.B, dtype=torch.int32).pin_memory(),
                    "acc_path": torch.zeros((cfg.B, cfg.D), dtype=torch.int32).pin_memory(),
                    "bonus": torch.zeros(cfg.B, dtype=torch.int32).pin_memory(),
                    "o": torch.zeros_like(out_all, device="cpu").pin_memory()}
        h2d = sum(t.numel() * t.element_size() for t in
                  [host_in["draft"], host_in["target"], host_in["ua"], host_in["ub"], host_in["q"], host_in["tree_kv"]])
        d2h = sum(t.numel() * t.element_size() for t in
                  [host_out["acc_len"], host_out["acc_path"], host_out["bonus"], host_out["o"]])

        # Two input sets alternate.  All of a step's inputs - logits, uniforms, queries, the tree
        # tokens' K/V rows (into a staging tensor) - go up on the copy stream, and the NEXT step's are
        # handed to it before this step's cycle is replayed, so that they travel under it: the one
        # host-to-device engine serves copies in the order they were issued (with the next logits
        # issued in front of this step's per-layer inputs a step took 2270 us; with the per-layer
        # inputs on the compute stream 1600 us).  The compute stream scatters the staged K/V rows into
        # the caches and replays the cycle.  Results go down on a third stream under the next step's
        # cycle, which writes the other set's output buffers; a set's next cycle waits for them.
        # Every step's copies, its own inputs included, lie inside the timed region.
        copy_stream = torch.cuda.Stream(device=dev)
        down_stream = torch.cuda.Stream(device=dev)
        ev_in = [torch.cuda.Event() for _ in range(2)]    # set j's logits have arrived
        ev_free = [torch.cuda.Event() for _ in range(2)]  # the cycle that read set j has finished
        ev_done = torch.cuda.Event()                      # the cycle's results are ready on the device
        ev_down = [torch.cuda.Event() for _ in range(2)]  # ... and set j's have reached the host buffers
        e2e_n = [0]                                       # steps of the running timed call

        def upload_inputs(j):
            s = sets[j]
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(ev_free[j])  # the cycle that read set j's buffers has finished
                s["q_all"].copy_(host_in["q"], non_blocking=True)
                tree_kv_dev[j].copy_(host_in["tree_kv"], non_blocking=True)
                s["draft"].copy_(host_in["draft"], non_blocking=True)
                s["target"].copy_(host_in["target"], non_blocking=True)
                s["ua"].copy_(host_in["ua"], non_blocking=True)
                s["ub"].copy_(host_in["ub"], non_blocking=True)
                ev_in[j].record(copy_stream)

        def e2e_step(i):
            j = i % 2
            s = sets[j]
            if i == 0:
                copy_stream.wait_stream(stream)  # nothing of the region starts before the region does
                down_stream.wait_stream(stream)
                upload_inputs(0)
            if i + 1 < e2e_n[0]:
                upload_inputs((i + 1) % 2)
            stream.wait_event(ev_in[j])   # this step's inputs are on the device
            for seq, (_, r) in enumerate(tree_rows):
                k_all[:, r:r + cfg.m].copy_(tree_kv_dev[j][:, 0, seq])
                v_all[:, r:r + cfg.m].copy_(tree_kv_dev[j][:, 1, seq])
            stream.wait_event(ev_down[j])  # the results of set j's last cycle have left the buffers this one writes
            graphs[j].replay()
            ev_free[j].record(stream)
            ev_done.record(stream)
            with torch.cuda.stream(down_stream):
                down_stream.wait_event(ev_done)
                host_out["acc_len"].copy_(s["buf"].acc_len, non_blocking=True)
                host_out["acc_path"].copy_(s["buf"].acc_path, non_blocking=True)
                host_out["bonus"].copy_(s["buf"].bonus_token, non_blocking=True)
                host_out["o"].copy_(s["out_all"], non_blocking=True)
                ev_down[j].record(down_stream)
            if i + 1 == e2e_n[0]:
                stream.wait_event(ev_down[j])  # the region ends when the last results are on the host

        e2e_steps = max(5, min(K, 50))
        e2e_n[0] = 3
        timed(e2e_step, 3)
        e2e_n[0] = e2e_steps
        ms_e2e = timed(e2e_step, e2e_steps)
    assert all(int(bb.status.item()) == 0 for bb in bufs), "device status raised during the timed region"

    us_cycle = ms_total * 1e3 / (K * world)
    us_attn = ms_attn * 1e3 / (attn_reps * cfg.n_layers)
    hbm_peak, tensor_peak, peak_kind = _peaks()
    achieved = attn_bytes / (us_attn * 1e-6) / 1e9
    # accepted length of the synthetic workload (tokens per cycle = accepted draft tokens + 1)
    acc = []
    with torch.cuda.stream(stream):
        for gr, z in zip(graphs, sets):
            gr.replay()
            stream.synchronize()
            acc.append(z["buf"].acc_len.float().mean().item())
    tau = float(np.mean(acc)) + 1.0

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- every floor of the attention call (one layer), and which one binds ---------------------------
    clk = clocks.summary()
    sm_hz = 1e6 * float(clk["sm_mhz"] or clk["sm_max_mhz"] or 1965)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    g_heads = cfg.Hq // cfg.Hkv
    keys = [int(L) + cfg.m for L in kv_len_h]
    tiles = [(n + 127) // 128 for n in keys]
    rows_padded = ((cfg.m * g_heads + 127) // 128) * 128 if cfg.m * g_heads <= 256 else 256 * math.ceil(cfg.m * g_heads / 256)
    flops_useful = float(sum(4 * cfg.m * cfg.Hq * n * cfg.d for n in keys))
    flops_issued = float(sum(4 * rows_padded * cfg.Hkv * 128 * t * cfg.d for t in tiles))
    exps = float(sum(cfg.m * cfg.Hq * n for n in keys))
    t_hbm = attn_bytes / (hbm_peak * 1e9) * 1e6
    t_tensor = flops_useful / (tensor_peak * 1e12) * 1e6
    t_tensor_issued = flops_issued / (tensor_peak * 1e12) * 1e6
    t_mufu = exps / (16.0 * sms * sm_hz) * 1e6
    floors = {"hbm": t_hbm, "tensor": t_tensor, "mufu": t_mufu}
    roofline_all = {
        "per": "one tree-attention call (one layer)", "measured_us": us_attn,
        "hbm_us": t_hbm, "tensor_us": t_tensor, "tensor_us_with_padding": t_tensor_issued, "mufu_us": t_mufu,
        "binding": max(floors, key=floors.get), "frac_of_binding_floor": max(floors.values()) / us_attn,
        "inputs": {"bytes": attn_bytes, "flops": flops_useful, "flops_issued": flops_issued, "exponentials": exps,
                   "hbm_gbs": hbm_peak, "bf16_tflops_sustained": tensor_peak,
                   "mufu": f"16 ex2 per clock per SM x {sms} SMs x {sm_hz / 1e6:.0f} MHz (sampled)"}}

    # ---- the vocabulary steps at this config, against the same HBM peak ----------------------------------
    us_expand, us_accept = breakdown["expand_x%d" % cfg.D], breakdown["accept"]
    expand_bytes = float(cfg.B) * cfg.R * cfg.V * 4
    parents = 0  # nodes (the root included) with a selected child, over the logit sets (mean)
    for z in sets:
        sp, si = z["buf"].sel_parent.cpu().numpy(), z["buf"].sel_index.cpu().numpy()
        parents += sum(len(set(int(q) for q, i in zip(sp[b], si[b]) if i >= 0)) for b in range(cfg.B))
    parents /= len(sets)
    if cfg.temperature > 0:
        accept_bytes_def = float(cfg.B * (cfg.m + 1) + parents) * cfg.V * 4   # every target row + the parents' draft rows
        accept_bytes_read = float(parents + cfg.B) * 2 * cfg.V * 4           # rows the kernels actually read
    else:
        accept_bytes_def = accept_bytes_read = float(cfg.B * (cfg.m + 1)) * cfg.V * 4
    step_rooflines = {
        "expand": {"us": us_expand, "calls": cfg.D, "algorithmic_bytes": expand_bytes,
                   "achieved_gbs": expand_bytes / (us_expand * 1e-6) / 1e9,
                   "frac_of_measured_hbm": expand_bytes / (us_expand * 1e-6) / 1e9 / hbm_peak},
        "accept": {"us": us_accept, "temperature": cfg.temperature, "parents_with_selected_children": parents,
                   "algorithmic_bytes": accept_bytes_def, "bytes_read": accept_bytes_read,
                   "frac_of_measured_hbm": accept_bytes_def / (us_accept * 1e-6) / 1e9 / hbm_peak,
                   "frac_of_measured_hbm_on_bytes_read": accept_bytes_read / (us_accept * 1e-6) / 1e9 / hbm_peak},
    }

    line = {
        "metric": METRIC, "value": us_cycle, "unit": "us", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_total / K, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 attention (fp32 accumulate), fp32 logits, fp64 node values", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "V": cfg.V, "k": cfg.k, "D": cfg.D, "m": cfg.m,
                   "n_layers": cfg.n_layers, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "d": cfg.d,
                   "kv_len": [int(x) for x in kv_len_h[:8]], "temperature": cfg.temperature,
                   "l2": f"inputs larger than L2: {cfg.n_layers} distinct KV layers "
                         f"({kv_bytes * cfg.n_layers / 1e6:.0f} MB) and {N_SETS} rotating logit sets",
                   "replicas": world, "synthetic_tau": tau},
        "clocks": clk,
        "per_replay_us": {"cycle": cycle_spread, "attention_layer": attn_spread, **breakdown_spread},
        "e2e": {"value": ms_e2e * 1e3 / (e2e_steps * world), "unit": "us", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h,
                "overlap": "the next step's inputs go up (copy stream, alternate input set) under this step's cycle, the results go down (third stream) under the next step's uploads"},
        "gpu_launches": buf.launches_per_cycle() * K,
        "roofline": {"kernel": "tree_attention_kernel + tree_attention_merge_kernel, one call per layer", "bound": "hbm",
                     "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
                     "peak_kind": f"of {peak_kind}", "traffic": None, "us_per_launch": us_attn,
                     "algorithmic_bytes_per_launch": attn_bytes},
    }
    if world == 1 and not args.no_cpu_baseline:
        total, parts, sample, cores = oracle_cycle_seconds(cfg)
        total1, parts1, _, _ = oracle_cycle_seconds(cfg, attn_samples=24, threads=1)
        line["cpu_baseline"] = {"value": total * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
                                "sample": sample, "parts_us": {k: v * 1e6 for k, v in parts.items()},
                                "single_thread": {"value": total1 * 1e6, "unit": "us", "cores": 1,
                                                  "parts_us": {k: v * 1e6 for k, v in parts1.items()}}}
    line["roofline"]["traffic"] = NCU_DRAM_BYTES_PER_LAUNCH.get(cfg.name)
    line["breakdown_us"] = breakdown  # each step replayed alone, rotating over the logit sets
    line["step_rooflines"] = step_rooflines
    line["roofline_all"] = roofline_all
    line["launch_floor"] = floor
    if world == 1 and not args.no_extras:
        line.update(side_measurements(e2, dev, stream, hbm_peak, args.extras))
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3_8b")
    ap.add_argument("--batch", type=int, default=0, help="override the number of sequences")
    ap.add_argument("--temperature", type=float, default=None, help="override the acceptance temperature")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the batched attention, expansion and acceptance side measurements")
    ap.add_argument("--extras-only", action="store_true", help="run only those side measurements (no bench line)")
    ap.add_argument("--extras", default="", help="comma-separated side measurements to run (default: all)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
