#!/usr/bin/env python
"""Benchmark of the WeDLM decoding step (reorder -> window attention -> confidence/commit).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3_batched] [--attn auto]
    python bench.py --impl reference ...        # the fp64 CPU oracle on a bounded sample

One "step" is one pass of the whole hot path over one batch of seeded synthetic inputs.  With
N > 1 (launched under torchrun) every rank runs the same-shaped batch drawn from its own seed
(weak scaling, sequences are independent: no collective on the data path) and rank 0 prints the
aggregate.  Prints ONE JSON line on stdout; progress goes to stderr.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "committed_tokens_per_s"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024

# DRAM traffic of the dominant kernel as a multiple of its algorithmic bytes
# (dram__bytes_read.sum + dram__bytes_write.sum from one ncu capture on a batch-40 case of the same
# shapes, which runs the same one-unit-per-CTA scheduling as the full batch: 705.5 MB against 704.0 MB;
# profiles/attn_tensor_kernel_cfg3_batch40.md gives the command).  Traffic grows with the tokens
# streamed, so the ratio is applied to the launch that is timed.  Missing = not captured.
NCU_TRAFFIC_RATIO = {"cfg3_batched:auto": 1.002, "cfg3_batched:tensor": 1.002}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the GPU works."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, device_index: int, period_s: float = 0.002):
        self.samples = []          # (t, sm_mhz, reasons_mask, tag)
        self.tag = "idle"
        self.period = period_s
        self._stop = threading.Event()
        self.ok = False
        self.max_mhz = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:          # pragma: no cover - depends on the box
            log("clock sampling unavailable:", repr(e))
        self.thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.time(), mhz, mask, self.tag))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.ok:
            self.thread.start()

    def stop(self):
        self._stop.set()
        if self.ok and self.thread.is_alive():
            self.thread.join(timeout=2)

    def summary(self, tag="timed"):
        """Median SM clock and the union of throttle reasons over the samples taken while `tag` was set
        (the headline line uses the samples inside the timed region of the main workload)."""
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        timed = [s for s in self.samples if s[3] == tag]
        use = timed if len(timed) >= 3 else [s for s in self.samples if s[3] != "idle"]
        if not use:
            use = self.samples
        mask = 0
        for s in use:
            mask |= s[2]
        reasons = [name for bit, name in self.REASONS.items() if mask & bit]
        return {"sm_mhz": statistics.median(s[1] for s in use), "sm_min_mhz": min(s[1] for s in use),
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(use),
                "samples_in_timed_region": len(timed)}


# ----------------------------------------------------------------------------------------------
# workload helpers
# ----------------------------------------------------------------------------------------------
def algorithmic_bytes(cfg, inp):
    """Bytes the method itself must move per step (one layer)."""
    elem = 2 if cfg.dtype == "bf16" else 4
    B, W = inp["filled"].shape
    kv_tokens = int(inp["prefix_len"].astype(np.int64).sum()) + B * W
    kv = kv_tokens * cfg.n_kv_heads * cfg.head_dim * 2 * elem             # K and V, prefix + window rows
    q_io = 2 * B * W * cfg.n_q_heads * cfg.head_dim * elem                # rotated q read + out write
    n_mask_rows = int((inp["filled"] == 0).sum())
    logits = n_mask_rows * cfg.vocab * elem
    # attention flops: QK^T and PV, 2 D flops per (row, key, query head) each; row i of sequence b sees P_b + i + 1 keys
    keys = int((inp["prefix_len"].astype(np.int64) * W + W * (W + 1) // 2).sum())
    flops = 4.0 * cfg.head_dim * cfg.n_q_heads * keys
    prefix_only = int(inp["prefix_len"].astype(np.int64).sum()) * cfg.n_kv_heads * cfg.head_dim * 2 * elem
    return {"attn_kernel": kv + q_io, "kv_stream": kv, "kv_prefix_only": prefix_only, "logits_stream": logits,
            "mask_rows": n_mask_rows, "attn_flops": flops}


def slice_batch(inp, n):
    out = {}
    for k, v in inp.items():
        out[k] = v if k in ("k_cache", "v_cache") else v[:n]
    return out


def oracle_step_time(cfg, inp, n_seqs):
    from oracle import wedlm_oracle as orc
    sub = slice_batch(inp, n_seqs)
    t0 = time.perf_counter()
    r = orc.step(sub, theta=cfg.rope_theta, conf_mode=cfg.conf_mode, tau=cfg.tau, lam=cfg.lam,
                 maxprob_thr=cfg.maxprob_thr, mask_token_id=cfg.mask_token_id, page_size=cfg.page_size)
    dt = time.perf_counter() - t0
    committed = int(sum(ps["committed_count"] for ps in r["per_seq"]))
    return dt, committed


# ----------------------------------------------------------------------------------------------
# reference arm: the oracle on host cores
# ----------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from workloads import get_config, make_step, BASE_SEED
    cfg = get_config(args.workload)
    inp = make_step(cfg, seed=BASE_SEED)
    cores = len(os.sched_getaffinity(0))
    # size the per-step sample so that the whole run stays within a few minutes
    t1, _ = oracle_step_time(cfg, inp, 1)
    budget_s = 150.0
    n = int(max(1, min(cfg.batch, budget_s / max(t1, 1e-3) / (args.steps + args.warmup))))
    for _ in range(args.warmup):
        oracle_step_time(cfg, inp, n)
    times, committed = [], 0
    for _ in range(args.steps):
        dt, c = oracle_step_time(cfg, inp, n)
        times.append(dt)
        committed = c
    total = sum(times)
    value = committed * args.steps / total if total > 0 else 0.0
    sample = f"first {n} of {cfg.batch} sequences of {cfg.name} per step (all heads, all mask rows)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------------------------
# product arm
# ----------------------------------------------------------------------------------------------
class Workload:
    """Device-resident inputs of one workload, with `n_copies` rotating copies of the large
    streams (cache, logits) when one copy would fit in L2, and one fresh copy of the small window
    state per iteration."""

    def __init__(self, name, seed, attn_impl, n_state, batch=None, temperature=0.0):
        import torch
        import paper_2512_22737_b200 as w
        from workloads import get_config, make_step
        self.cfg = get_config(name)
        if batch:
            self.cfg = self.cfg.replace(batch=batch)
        t0 = time.time()
        self.inp = make_step(self.cfg, seed=seed)
        log(f"[{name}] inputs drawn in {time.time() - t0:.1f}s")
        inp = self.inp
        self.bytes = algorithmic_bytes(self.cfg, inp)
        big = inp["k_cache"].nbytes + inp["v_cache"].nbytes + inp["logits"].nbytes
        self.n_copies = 1 if big > 2 * L2_BYTES else int(np.ceil(3 * L2_BYTES / big)) + 1
        self.c = w.config_for(self.cfg, max_pages_per_seq=inp["block_table"].shape[1],
                              num_pages=inp["k_cache"].shape[0], max_prefix_len=int(inp["prefix_len"].max()),
                              attn_impl=attn_impl, sample_temperature=temperature, sample_seed=seed)
        self.step = w.DecodeStep(self.c)
        self.static = {k: w.to_device(inp[k]) for k in ("q", "k", "v", "block_table")}
        self.big = [{k: (w.to_device(inp[k]) if i == 0 else None) for k in ("k_cache", "v_cache", "logits")}
                    for i in range(self.n_copies)]
        for i in range(1, self.n_copies):
            for k in ("k_cache", "v_cache", "logits"):
                self.big[i][k] = self.big[0][k].clone()
        self.state0 = {k: w.to_device(inp[k]) for k in ("filled", "window_tokens", "prefix_len")}
        self.states = [{k: v.clone() for k, v in self.state0.items()} for _ in range(n_state)]
        self.it = 0
        self.committed_per_step = None
        torch.cuda.synchronize()

    def reset_states(self):
        for s in self.states:
            for k, v in self.state0.items():
                s[k].copy_(v)
        self.it = 0

    def run_step(self, profile_events=None):
        import paper_2512_22737_b200 as w
        big = self.big[self.it % self.n_copies]
        st = self.states[self.it % len(self.states)]
        self.it += 1
        d = dict(self.static)
        d.update(big)
        d.update(st)
        s = self.step
        s.reorder(d["filled"], d["window_tokens"], d["prefix_len"])
        if profile_events is not None:
            w.wedlm_profile_next_attn(*profile_events)
        s.attention(d["q"], d["k"], d["v"], d["k_cache"], d["v_cache"], d["block_table"], d["prefix_len"])
        s.confidence_commit(d["logits"], d["window_tokens"], d["filled"], d["prefix_len"])


def time_workload(wl, steps, warmup, sampler=None, tag="timed", min_region_s=1.0, max_blocks=2000):
    """`warmup` untimed steps, then blocks of exactly `steps` steps, each block bracketed by CUDA events on the
    launching stream, repeated back to back until the timed blocks add up to `min_region_s` (steady state: the
    clocks have settled under the load).  The window state is restored between blocks, outside the events.
    Returns a dict: mean / median / best ms per step over the blocks, the mean duration of the attention kernel
    (events placed inside wedlm_window_attn around that kernel), commits per step, launches per step."""
    import torch
    import paper_2512_22737_b200 as w
    wl.reset_states()
    for _ in range(warmup):
        wl.run_step()
    torch.cuda.synchronize()
    committed = int(wl.step.committed_count.sum().item())
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:       # create the handles outside the timed region
        a.record()
        b.record()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    block_ms, attn_ms_sum, launches = [], 0.0, 0
    if sampler:
        sampler.tag = tag
    while not block_ms or (sum(block_ms) < min_region_s * 1e3 and len(block_ms) < max_blocks):
        wl.reset_states()
        l0 = w.wedlm_launch_count()
        start.record()
        for i in range(steps):
            wl.run_step(profile_events=evs[i])
        stop.record()
        torch.cuda.synchronize()
        launches = w.wedlm_launch_count() - l0
        block_ms.append(start.elapsed_time(stop))
        attn_ms_sum += sum(a.elapsed_time(b) for a, b in evs)
    if sampler:
        sampler.tag = "other"
    n_blocks = len(block_ms)
    per_step = sorted(x / steps for x in block_ms)
    return {"ms": sum(block_ms) / (n_blocks * steps), "ms_median": statistics.median(per_step), "ms_best": per_step[0],
            "attn_ms": attn_ms_sum / (n_blocks * steps), "committed": committed, "launches": launches,
            "blocks": n_blocks, "region_s": sum(block_ms) * 1e-3}


def time_graph(wl, steps, warmup, min_region_s=0.25):
    """The same step captured once into a CUDA graph (the window state is restored from pristine copies
    inside the graph, three small device copies) and replayed: launch overhead removed.  Uses the first
    copy of the large streams, so workloads that fit in L2 run warm here."""
    import torch
    d = dict(wl.static)
    d.update(wl.big[0])
    st = wl.states[0]
    d.update(st)
    s = wl.step

    def body():
        for k, v in wl.state0.items():
            st[k].copy_(v)
        s.reorder(d["filled"], d["window_tokens"], d["prefix_len"])
        s.attention(d["q"], d["k"], d["v"], d["k_cache"], d["v_cache"], d["block_table"], d["prefix_len"])
        s.confidence_commit(d["logits"], d["window_tokens"], d["filled"], d["prefix_len"])

    body()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        body()
    for _ in range(warmup):
        graph.replay()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total, n = 0.0, 0
    while n == 0 or (total < min_region_s * 1e3 and n < 2000 * steps):
        start.record()
        for _ in range(steps):
            graph.replay()
        stop.record()
        torch.cuda.synchronize()
        total += start.elapsed_time(stop)
        n += steps
    return total / n


def time_e2e(wl, steps, warmup, sampler=None, mode="lmhead", hidden=4096, lm_head=None):
    """The same step through the library's calls for step inputs that live in HOST memory: every iteration sends
    the window state, block table and q/k/v from page-locked host buffers, runs reorder -> attention ->
    confidence/commit and brings the commit results and the new window state back.  The KV cache is resident
    device state, as in a serving engine.
      mode "lmhead": wedlm_step_host_lmhead - the hidden states of the window rows come from the host, the output
                     embedding is resident and the LM head runs inside the step (what a serving loop hands over);
      mode "logits": wedlm_step_host - the [B,W,V] logits themselves come from the host (only the rows the step
                     reads are sent); this leg measures the host link."""
    import torch
    import paper_2512_22737_b200 as w
    inp = wl.inp
    names = ["filled", "window_tokens", "prefix_len", "block_table", "q", "k", "v"] + (["logits"] if mode == "logits" else [])
    src = {}
    for k in names:
        a = inp[k]
        src[k] = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
    host = {k: src[k].clone().pin_memory() for k in names}
    state = ("filled", "window_tokens", "prefix_len")
    B, W = inp["filled"].shape
    ct = torch.empty(B, W, dtype=torch.int32).pin_memory()
    cc = torch.empty(B, dtype=torch.int32).pin_memory()
    fc = torch.empty(B, dtype=torch.int32).pin_memory()
    big = wl.big[0]
    elem = 2 if wl.cfg.dtype == "bf16" else 4
    n_mask_rows = int((inp["filled"] == 0).sum())
    small = sum(host[k].numel() * host[k].element_size() for k in names if k != "logits")
    d2h = sum(t.numel() * t.element_size() for t in (ct, cc, fc)) + sum(host[k].numel() * host[k].element_size() for k in state)
    if mode == "logits":
        ws = torch.empty(w.wedlm_step_host_workspace_bytes(wl.c), dtype=torch.uint8, device="cuda")
        h2d = small + n_mask_rows * wl.cfg.vocab * elem

        def call():
            w.wedlm_step_host(wl.c, host["filled"], host["window_tokens"], host["prefix_len"], None, None, host["block_table"],
                              host["q"], host["k"], host["v"], host["logits"], big["k_cache"], big["v_cache"], ct, cc, fc, ws,
                              wl.step.status)
    else:
        g = torch.Generator().manual_seed(251222737)
        h_hid = torch.randn(B, W, hidden, generator=g).to(torch.bfloat16).pin_memory()
        ws = torch.empty(w.wedlm_step_host_lmhead_workspace_bytes(wl.c, hidden), dtype=torch.uint8, device="cuda")
        h2d = small + h_hid.numel() * 2

        def call():
            w.wedlm_step_host_lmhead(wl.c, host["filled"], host["window_tokens"], host["prefix_len"], None, None,
                                     host["block_table"], host["q"], host["k"], host["v"], h_hid, lm_head, None, 0.0,
                                     big["k_cache"], big["v_cache"], ct, cc, fc, ws, wl.step.status)

    def one():
        for k in state:                       # the step updates the window state in place: start from the same one
            host[k].copy_(src[k])
        call()
        torch.cuda.synchronize()              # the caller reads the commits before it can build the next step

    for _ in range(warmup):
        one()
    torch.cuda.synchronize()
    if sampler:
        sampler.tag = "e2e_" + mode
    t0 = time.perf_counter()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        one()
    stop.record()
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3 / steps
    if sampler:
        sampler.tag = "other"
    ms = max(start.elapsed_time(stop) / steps, wall_ms)
    committed = int(cc.sum().item())
    return ms, committed, h2d, d2h


def rank_seed(rank: int) -> int:
    """Every rank draws its own batch of the same shape (weak scaling over independent sequences)."""
    from workloads import BASE_SEED
    return BASE_SEED + rank


def reduce_over_ranks(times_ms, counts, device):
    """Job-level figures from per-rank ones: MAX over ranks of every time, SUM over ranks of every
    count.  Works on any backend (NCCL on the GPUs, gloo in the CPU tests); a single process returns
    its own values."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    c = torch.tensor(list(counts), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [float(x) for x in c.tolist()]


def tensor_peaks():
    """Measured bf16 GEMM throughput on this machine (burst and sustained), or the stated fallback."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return float(p["bf16_tflops"]), float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "measured"
    except Exception:
        return 1590.0, 1400.0, "fallback"


def run_product(args):
    import torch
    import torch.distributed as dist
    from paper_2512_22737_b200 import build as b
    from workloads import BASE_SEED

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        b.build()
    if world > 1:
        dist.barrier()
    import paper_2512_22737_b200 as w
    w.load_library()

    sampler = ClockSampler(local) if rank == 0 else None
    n_state = max(args.steps, args.warmup)
    wl = Workload(args.workload, rank_seed(rank), args.attn, n_state, args.batch, args.temperature)
    if sampler:
        sampler.start()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    t = time_workload(wl, args.steps, args.warmup, sampler, min_region_s=args.min_seconds)
    barrier()
    (ms, ms_median, ms_best, attn_ms), (committed_total,) = reduce_over_ranks(
        [t["ms"], t["ms_median"], t["ms_best"], t["attn_ms"]], [t["committed"]], "cuda")
    launches = t["launches"]
    assert int(wl.step.status.item()) == 0, "device status word set during the benchmark"

    # end to end from host buffers: hidden states in (LM head inside the step), and the logits-from-host variant
    e2e = {"lmhead": None, "logits": None}
    if not args.no_e2e and wl.cfg.dtype == "bf16":
        hidden = 4096
        g = torch.Generator(device="cuda").manual_seed(rank_seed(rank))
        lm_head = (torch.randn(wl.cfg.vocab, hidden, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
        e2e["lmhead"] = time_e2e(wl, max(3, min(args.steps, 10)), 3, sampler, "lmhead", hidden, lm_head)
        del lm_head
        torch.cuda.empty_cache()
        e2e["logits"] = time_e2e(wl, max(3, min(args.steps, 10)), 3, sampler, "logits")
    elif not args.no_e2e:
        e2e["logits"] = time_e2e(wl, max(3, min(args.steps, 10)), 3, sampler, "logits")
    e2e_json = {}
    for mode, r in e2e.items():
        r = r or (float("nan"), 0, 0, 0)
        (e_ms,), (e_commit,) = reduce_over_ranks([r[0]], [r[1]], "cuda")
        e2e_json[mode] = {"value": (e_commit / (e_ms * 1e-3)) if e_ms == e_ms else None, "unit": UNIT,
                          "ms_per_step": e_ms if e_ms == e_ms else None, "h2d_bytes_per_step": r[2], "d2h_bytes_per_step": r[3]}
    e2e_json["lmhead"]["call"] = "wedlm_step_host_lmhead: hidden states [B,W,4096] from pinned host memory, output embedding resident"
    e2e_json["logits"]["call"] = "wedlm_step_host: logits rows of the mask slots from pinned host memory"

    graph_ms = time_graph(wl, args.steps, args.warmup) if world == 1 else None
    peak, peak_kind = measured_peaks()
    tf_burst, tf_sustained, tf_kind = tensor_peaks()
    others, extras, cpu = {}, {}, None
    if rank == 0 and world == 1 and not args.no_extras:
        for name in ("cfg2_qwen_b1", "cfg4_long"):
            if name == args.workload:
                continue
            try:
                o = Workload(name, BASE_SEED, args.attn, n_state)
                ot = time_workload(o, args.steps, args.warmup, sampler, tag=name, min_region_s=0.4 * args.min_seconds)
                ob = o.bytes
                gms = time_graph(o, args.steps, args.warmup)
                a_ms = ot["attn_ms"]
                others[name] = {
                    "ms_per_step": ot["ms"], "ms_per_step_median": ot["ms_median"], "ms_per_step_best": ot["ms_best"],
                    "timed_region_s": ot["region_s"], "timed_blocks": ot["blocks"],
                    "committed_tokens_per_s": ot["committed"] / (ot["ms"] * 1e-3),
                    "cuda_graph_ms_per_step": gms, "cuda_graph_l2": "cold" if o.n_copies == 1 else "warm",
                    "attn_kernel_ms": a_ms, "attn_kernel_GBps": ob["attn_kernel"] / (a_ms * 1e-3) / 1e9,
                    "rotating_copies": o.n_copies, "clocks": sampler.summary(name) if sampler else None,
                    # the attention kernel against both roofs (this shape sits on the ridge)
                    "roofline": {
                        "kernel": "window attention", "kernel_ms": a_ms,
                        "hbm": {"algorithmic_bytes": ob["attn_kernel"], "achieved_GBps": ob["attn_kernel"] / (a_ms * 1e-3) / 1e9,
                                "peak_GBps": peak, "frac": ob["attn_kernel"] / (a_ms * 1e-3) / 1e9 / peak,
                                "frac_of_nominal_8TBps": ob["attn_kernel"] / (a_ms * 1e-3) / 1e9 / 8000.0},
                        "tensor": {"flops": ob["attn_flops"], "achieved_TFLOPs": ob["attn_flops"] / (a_ms * 1e-3) / 1e12,
                                   "peak_TFLOPs_burst": tf_burst, "peak_TFLOPs_sustained": tf_sustained,
                                   "frac_of_burst": ob["attn_flops"] / (a_ms * 1e-3) / 1e12 / tf_burst,
                                   "frac_of_sustained": ob["attn_flops"] / (a_ms * 1e-3) / 1e12 / tf_sustained,
                                   "peak_kind": tf_kind}},
                }
                del o
                torch.cuda.empty_cache()
            except Exception as e:      # pragma: no cover
                others[name] = {"error": repr(e)}
        # short legs of the other parts of the library, so that every measured claim has a line here
        for key, fn in (("lmhead", lambda: measure_lmhead(args.steps, args.warmup)),
                        ("dual_stream", lambda: measure_dual_stream(["ds_4k"], args.attn, args.steps, args.warmup)),
                        ("cfg5_loop", lambda: measure_loop_short(args))):
            try:
                if sampler:
                    sampler.tag = key
                extras[key] = fn()
                if sampler:
                    extras[key]["clocks"] = sampler.summary(key)
                    sampler.tag = "other"
                torch.cuda.empty_cache()
            except Exception as e:      # pragma: no cover
                extras[key] = {"error": repr(e)}
    if sampler:
        sampler.stop()
    if rank == 0 and world == 1 and not args.no_cpu:
        cores = len(os.sched_getaffinity(0))
        # bounded sample: as many sequences of the batch as fit in about 20 s of oracle time
        n_probe = min(wl.cfg.batch, 4)
        dt_probe, _ = oracle_step_time(wl.cfg, wl.inp, n_probe)
        n_s = int(max(n_probe, min(wl.cfg.batch, 20.0 / max(dt_probe / n_probe, 1e-3))))
        log(f"timing the oracle on {n_s} sequences ...")
        dt, c = oracle_step_time(wl.cfg, wl.inp, n_s)
        cpu = {"value": c / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"one step over the first {n_s} of {wl.cfg.batch} sequences of {wl.cfg.name} "
                         f"({dt:.1f}s of CPU wall time)"}

    if rank == 0:
        bts = wl.bytes
        achieved = bts["attn_kernel"] / (attn_ms * 1e-3) / 1e9
        key = f"{wl.cfg.name}:{args.attn}"
        clocks = sampler.summary("timed") if sampler else None
        head_e2e = e2e_json["lmhead"] if e2e_json["lmhead"]["value"] is not None else e2e_json["logits"]
        line = {
            "metric": METRIC, "value": committed_total / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if wl.cfg.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": wl.cfg.name if not args.batch else f"{wl.cfg.name}@batch{args.batch}", "batch_per_gpu": wl.cfg.batch, "window": wl.cfg.window,
                       "prefix_tokens_per_gpu": int(wl.inp["prefix_len"].sum()), "attn_impl": args.attn,
                       "l2": "inputs_exceed_l2" if wl.n_copies == 1 else f"rotating_{wl.n_copies}_copies",
                       "committed_tokens_per_step": committed_total,
                       "sample": "argmax" if args.temperature <= 0 else f"gumbel_max_T{args.temperature:g}",
                       "kv_stream_bytes": bts["kv_stream"], "logits_stream_bytes": bts["logits_stream"]},
            # steady state: blocks of `steps` steps repeated back to back until the timed region is long enough for the
            # clocks to settle; ms_per_step (and value) is the mean over the whole region
            "timing": {"timed_blocks": t["blocks"], "timed_region_s": t["region_s"], "steps_per_block": args.steps,
                       "ms_per_step_median": ms_median, "ms_per_step_best": ms_best,
                       "ms_x_sm_mhz": (ms * clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None},
            "clocks": clocks,
            "e2e": head_e2e,
            "e2e_logits_host": e2e_json["logits"],
            "gpu_launches": int(launches),
            "cuda_graph": None if graph_ms is None else {"ms_per_step": graph_ms, "value": committed_total / (graph_ms * 1e-3),
                                                         "note": "same step replayed from one captured graph"},
            "roofline": {"bound": "hbm", "kernel": "window attention", "achieved": achieved, "peak": peak,
                         "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_nominal_8TBps": achieved / 8000.0,
                         "traffic": (NCU_TRAFFIC_RATIO[key] * bts["attn_kernel"] if key in NCU_TRAFFIC_RATIO and not args.batch else None),
                         "traffic_note": "ncu dram bytes of a batch-40 capture scaled by algorithmic bytes",
                         "kernel_ms": attn_ms,
                         "algorithmic_bytes": bts["attn_kernel"],
                         "bytes_definition": "K and V of every cached prefix token AND of the staged window rows (4096 B per token), "
                                             "plus the rotated q read and the output write",
                         "frac_prefix_tokens_only": bts["kv_prefix_only"] / (attn_ms * 1e-3) / 1e9 / peak},
            "step_hbm": {"note": "whole step: K/V and logits streams plus q/out, against the same measured peak",
                         "algorithmic_bytes": bts["attn_kernel"] + bts["logits_stream"],
                         "achieved": (bts["attn_kernel"] + bts["logits_stream"]) / (ms * 1e-3) / 1e9, "unit": "GB/s",
                         "frac": (bts["attn_kernel"] + bts["logits_stream"]) / (ms * 1e-3) / 1e9 / peak},
            "cpu_baseline": cpu,
            "other_workloads": others,
        }
        line.update(extras)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


# ----------------------------------------------------------------------------------------------
# end-to-end streaming decode loop (the 4-layer configuration); not the default bench line
# ----------------------------------------------------------------------------------------------
def measure_loop_short(args):
    """The end-to-end loop in a form short enough for the default line: 256 new tokens per sequence at the
    calibrated tilt lse + 8, streaming commits, W = 16 against the same harness at W = 2 and W = 1, and W = 16 once
    more with the LM head fused into the confidence call."""
    import types
    a = types.SimpleNamespace(**vars(args))
    a.loop_new_tokens, a.loop_windows, a.loop_block_windows, a.loop_fused_windows = 256, [16, 2, 1], [], [16]
    a.loop_tilts, a.loop_eager = [("lse", 8.0)], False
    line = measure_loop(a)
    by_w = {r["window"]: r for r in line["results"] if r["lm_head"] != "fused"}
    out = {"config": line["config"], "results": line["results"], "unit": "generated tokens/s"}
    if 16 in by_w and 1 in by_w:
        out["speedup_w16_over_w1"] = by_w[16]["tokens_per_s"] / by_w[1]["tokens_per_s"]
    if 16 in by_w and 2 in by_w:
        out["speedup_w16_over_w2"] = by_w[16]["tokens_per_s"] / by_w[2]["tokens_per_s"]
    return out


def run_loop(args):
    print(json.dumps(measure_loop(args)), flush=True)
    return 0


def measure_loop(args):
    """Random-init 4-layer model of Qwen3-8B width, batch 16, 512-token prompt, 1024 new tokens per
    sequence, LM-head logits tilted toward a seeded target sequence.  Generated tokens/s, steps and
    p_cache (Eq. 4) for W = 16 against the same harness at W = 1 and W = 2, for every tilt."""
    import torch
    from paper_2512_22737_b200 import build as b
    from paper_2512_22737_b200.loop import StreamingDecoder
    from workloads.model import QWEN_4L, make_prompts_and_targets
    b.build()
    torch.cuda.set_device(0)
    m = QWEN_4L
    B, P, N = args.loop_batch, 512, args.loop_new_tokens
    g = torch.Generator(device="cuda").manual_seed(251222737)
    H, F = m.hidden, m.ffn

    def mat(*shape):
        return (torch.randn(*shape, generator=g, device="cuda", dtype=torch.float32) * m.init_std).to(torch.bfloat16)

    class DeviceWeights(dict):
        pass
    wts = DeviceWeights(embed=mat(m.vocab, H), lm_head=mat(H, m.vocab), norm_f=torch.ones(H, device="cuda", dtype=torch.bfloat16))
    for l in range(m.n_layers):
        wts[f"l{l}.norm1"] = torch.ones(H, device="cuda", dtype=torch.bfloat16)
        wts[f"l{l}.norm2"] = torch.ones(H, device="cuda", dtype=torch.bfloat16)
        wts[f"l{l}.wq"] = mat(H, m.n_q_heads * m.head_dim)
        wts[f"l{l}.wk"] = mat(H, m.n_kv_heads * m.head_dim)
        wts[f"l{l}.wv"] = mat(H, m.n_kv_heads * m.head_dim)
        wts[f"l{l}.wo"] = mat(m.n_q_heads * m.head_dim, H)
        wts[f"l{l}.wg"] = mat(H, F)
        wts[f"l{l}.wu"] = mat(H, F)
        wts[f"l{l}.wd"] = mat(F, H)
    pt = make_prompts_and_targets(m, B, P, N)
    results = []
    lse0 = None
    runs = [(W, "streaming", False) for W in args.loop_windows] + [(W, "block", False) for W in args.loop_block_windows] + \
           [(W, "streaming", True) for W in args.loop_fused_windows]
    lm_head_vh = wts["lm_head"].t().contiguous() if args.loop_fused_windows else None
    for W, mode, fused in runs:
        for tilt_name, tilt in args.loop_tilts:
            # a short untimed run of the same geometry first: the first GEMMs of a new shape and the first capture
            # pay one-off library set-up that is no part of the decode rate
            for phase_tokens in (min(8, N), N):
                dec = StreamingDecoder(m, {}, batch=B, window=W, max_total_len=P + N, tau=args.loop_tau, lam=args.loop_lambda,
                                       tilt=0.0, target=pt["target"], commit_mode=mode, fused_lm_head=fused)
                dec.wt = wts
                dec.lm_head_vh = lm_head_vh
                dec.prefill(pt["prompt"])
                if lse0 is None:                    # log-sum-exp of the untilted logits, measured once
                    dec.start(N)
                    lg, _ = dec.forward()
                    lse0 = float(torch.logsumexp(lg[:, 0].float(), dim=-1).mean().item())
                dec.tilt = tilt if tilt_name == "literal" else lse0 + tilt
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                out = dec.generate(phase_tokens, use_graph=not args.loop_eager)
                torch.cuda.synchronize()
                dt = time.perf_counter() - t0
                if phase_tokens != N:
                    del dec
            n_gen = sum(len(y) for y in out["y"])
            on_target = sum(int(out["y"][bb] == pt["target"][bb, P:P + N].tolist()) for bb in range(B))
            results.append({"window": W, "commit": mode, "lm_head": "fused" if fused else "gemm+logits",
                            "replay": "eager" if args.loop_eager else "cuda_graph",
                            "tilt": f"{tilt_name}+{tilt:g}", "tokens_per_s": n_gen / out.get("decode_s", dt), "seconds": dt,
                            "decode_seconds": out.get("decode_s", dt), "capture_seconds": out.get("capture_s", 0.0),
                            "steps": out["steps"], "tokens_per_step_per_seq": n_gen / B / max(out["steps"], 1),
                            "p_cache": out["p_cache"], "sequences_equal_to_target": on_target})
            log(results[-1])
            del dec
            torch.cuda.empty_cache()
    line = {"metric": "generated_tokens_per_s", "unit": "tokens/s", "n_gpus": 1, "data": "synthetic", "dtype": "bf16",
            "config": {"workload": "cfg5_loop", "batch": B, "prompt": P, "new_tokens": N, "layers": m.n_layers,
                       "tau": args.loop_tau, "lambda": args.loop_lambda,
                       "hidden": H, "lse_of_untilted_logits": lse0,
                       "timing": "host wall clock of the decode loop (graph replays with the per-step read-back of commits), after one short untimed run of the same geometry; capturing the step once is timed apart (capture_seconds); eager runs time generate() whole"},
            "results": results}
    del wts, lm_head_vh
    return line


def run_lmhead(args):
    print(json.dumps(measure_lmhead(args.steps, args.warmup)), flush=True)
    return 0


def measure_lmhead(steps, warmup):
    """LM head + confidence/commit, hidden 4096 and vocabulary 151 936, at two row counts: 16 x 16 (the shape of a
    small serving batch) and 64 x 32 (the headline workload's windows, 30 % of the slots already filled).  The fused
    call (mask rows gathered, logits kept in tensor memory) against a library GEMM over all rows that writes bf16
    logits followed by the streaming confidence call."""
    import torch
    from paper_2512_22737_b200 import build as b
    b.build()
    import paper_2512_22737_b200 as w
    torch.cuda.set_device(0)
    V, H = 151936, 4096
    torch.manual_seed(0)
    emb = (torch.randn(V, H, device="cuda") * 0.02).to(torch.bfloat16)
    emb_hv = emb.t().contiguous()
    shapes = {}
    for B, W in ((16, 16), (64, 32)):
        hid = torch.randn(B, W, H, device="cuda").to(torch.bfloat16)
        c = w.make_config(batch=B, window=W, n_q_heads=32, n_kv_heads=8, head_dim=128, max_pages_per_seq=4, num_pages=64,
                          vocab=V, dtype="bf16", mask_token_id=V - 1, max_prefix_len=16)
        step = w.DecodeStep(c)
        filled = (torch.rand(B, W, device="cuda") < 0.3).to(torch.uint8)
        tok = torch.zeros(B, W, dtype=torch.int32, device="cuda")
        pl = torch.full((B,), 16, dtype=torch.int32, device="cuda")
        step.reorder(filled, tok, pl)
        mask_rows = int(B * W - step.n_filled.sum().item())
        ws = torch.empty(w.wedlm_lmhead_confidence_workspace_bytes(c, H), dtype=torch.uint8, device="cuda")

        def fused(f, t, p):
            w.wedlm_lmhead_confidence_commit(c, hid, emb, None, 0.0, step.perm, step.n_filled, step.n_commit, t, f, p, None,
                                             None, step.argmax, step.maxprob, step.entropy, step.lse, step.committed_tokens,
                                             step.committed_count, step.filled_count, ws, step.status)

        def unfused(f, t, p):
            step.confidence_commit((hid @ emb_hv).contiguous(), t, f, p)

        out = {}
        for name, fn in (("fused", fused), ("gemm_then_confidence", unfused)):
            ts = []
            for _ in range(warmup + steps):
                f, t, p = filled.clone(), tok.clone(), pl.clone()
                a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn(f, t, p)
                e.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(e))
            ts = ts[warmup:]
            out[name] = {"ms_min": min(ts), "ms_median": statistics.median(ts)}
        assert int(step.status.item()) == 0
        # the tensor cores run whole 256-row chunks of the gathered mask rows; the flops that count are the mask rows'
        chunks = (mask_rows + 255) // 256
        t = out["fused"]["ms_median"] * 1e-3
        out.update({"rows": B * W, "mask_rows": mask_rows, "flops_mask_rows": 2 * mask_rows * H * V,
                    "flops_tiles": 2 * chunks * 256 * H * V,
                    "fused_TFLOPs_mask_rows": 2 * mask_rows * H * V / t / 1e12,
                    "fused_TFLOPs_tiles": 2 * chunks * 256 * H * V / t / 1e12,
                    "fused_weight_stream_GBps": V * H * 2 / t / 1e9})
        shapes[f"{B}x{W}"] = out
        del hid, ws, step
    return {"metric": "lm_head_confidence_ms", "unit": "ms", "n_gpus": 1, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "lmhead", "hidden": H, "vocab": V, "filled_fraction": 0.3},
            "weight_bytes": V * H * 2, "shapes": shapes}


# ----------------------------------------------------------------------------------------------
# Dual-Stream Masking training forward (Section 4.2): attention over the two-stream input
# ----------------------------------------------------------------------------------------------
def run_dual_stream(args):
    print(json.dumps(measure_dual_stream(args.ds_configs, args.attn, args.steps, args.warmup)), flush=True)
    return 0


def measure_dual_stream(ds_configs, attn, steps, warmup):
    import torch
    from paper_2512_22737_b200 import build as b
    from workloads import DS_CONFIGS, make_dual_stream
    b.build()
    import paper_2512_22737_b200 as w
    torch.cuda.set_device(0)
    out = {}
    for name in ds_configs:
        c = DS_CONFIGS[name]
        inp = make_dual_stream(c)
        cfg = w.make_config(batch=c.n_seq, window=c.block, n_q_heads=c.n_q_heads, n_kv_heads=c.n_kv_heads,
                            head_dim=c.head_dim, page_size=c.page_size, vocab=c.vocab, dtype=c.dtype,
                            rope_theta=c.rope_theta, mask_token_id=c.mask_token_id, attn_impl=attn)
        N, K, L, B, Lp = c.n_seq, c.n_blocks, c.seq_len, c.block, c.padded_len
        i32 = dict(dtype=torch.int32, device="cuda")
        tokens, masked = w.to_device(inp["tokens"]), w.to_device(inp["masked"])
        x, pin = torch.empty(N, 2, Lp, **i32), torch.empty(N, 2, Lp, **i32)
        q, k, v = (w.to_device(inp[t]) for t in ("q", "k", "v"))
        o = torch.empty_like(q)
        ws = torch.empty(w.wedlm_dual_stream_workspace_bytes(cfg, K), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, **i32)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")       # larger than L2
        ts, launches0 = [], w.wedlm_launch_count()
        for it in range(warmup + steps):
            flush.fill_(it & 0xff)
            a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            w.wedlm_dual_stream_construct(cfg, K, L, tokens, masked, x, pin)
            w.wedlm_dual_stream_attn(cfg, K, q, k, v, pin, o, ws, status)
            e.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(e))
        assert int(status.item()) == 0
        launches = (w.wedlm_launch_count() - launches0) // (warmup + steps)
        ts = ts[warmup:]
        ms = statistics.median(ts)
        # visible keys per row: k*B + r + 1, both streams; QK^T and PV are 2*D flops per (row, key, head) each
        keys = 2 * sum((i // B) * B + (i % B) + 1 for i in range(L))
        flops = 4.0 * c.head_dim * c.n_q_heads * keys * N
        elem = 2 if c.dtype == "bf16" else 4
        io_bytes = N * 2 * Lp * (2 * c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim * elem      # q, out, k, v once
        out[name] = {"ms_median": ms, "ms_min": min(ts), "tokens_per_s": N * L / (ms * 1e-3),
                     "attention_TFLOPs": flops / (ms * 1e-3) / 1e12, "flops": flops, "io_bytes": io_bytes,
                     "launches_per_forward": int(launches), "seq_len": L, "block": B, "n_seq": N}
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak, kind = float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        peak, kind = 1590.0, "fallback"
    first = out[ds_configs[0]]
    line = {"metric": "dual_stream_attention_tokens_per_s", "value": first["tokens_per_s"], "unit": "tokens/s", "n_gpus": 1,
            "dtype": "bf16", "data": "synthetic", "higher_is_better": True,
            "config": {"workload": ds_configs[0], "l2": "flushed between iterations", "attn_impl": attn},
            "roofline": {"bound": "tensor", "achieved": first["attention_TFLOPs"], "peak": peak, "peak_kind": kind,
                         "unit": "TFLOP/s", "frac": first["attention_TFLOPs"] / peak, "traffic": None},
            "results": out}
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="product", choices=["product", "reference"])
    ap.add_argument("--workload", default="cfg3_batched")
    ap.add_argument("--attn", default="auto", choices=["auto", "generic", "tensor"])
    ap.add_argument("--no-extras", action="store_true", help="skip the secondary workloads")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the oracle timing (profiling runs)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (profiling runs)")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="blocks of --steps steps are repeated until the timed region is at least this long")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="Sample() temperature of the step workloads (0 = arg-max, the headline configuration)")
    ap.add_argument("--ds-configs", type=lambda s: s.split(","), default=["ds_4k", "ds_8k"],
                    help="dual-stream training-forward shapes timed by --workload dual_stream")
    ap.add_argument("--loop-batch", type=int, default=16)
    ap.add_argument("--loop-new-tokens", type=int, default=1024)
    ap.add_argument("--loop-windows", type=lambda s: [int(x) for x in s.split(",")], default=[16, 2, 1])
    ap.add_argument("--loop-fused-windows", type=lambda s: [int(x) for x in s.split(",") if x], default=[],
                    help="windows also run with the LM head fused into the confidence call")
    ap.add_argument("--loop-eager", action="store_true",
                    help="launch every step kernel by kernel instead of replaying one captured CUDA graph")
    ap.add_argument("--loop-tau", type=float, default=0.3)
    ap.add_argument("--loop-lambda", type=float, default=0.1)
    ap.add_argument("--loop-block-windows", type=lambda s: [int(x) for x in s.split(",") if x], default=[16],
                    help="windows also run with the block-wise commit rule (the baseline of Fig. 3c)")
    ap.add_argument("--loop-tilts", type=lambda s: [(t.split(":")[0], float(t.split(":")[1])) for t in s.split(",")],
                    default=[("literal", 2.0), ("literal", 4.0), ("literal", 8.0), ("lse", 2.0), ("lse", 4.0), ("lse", 8.0)])
    args = ap.parse_args()
    if args.workload == "cfg5_loop":
        return run_loop(args)
    if args.workload == "lmhead":
        return run_lmhead(args)
    if args.workload == "dual_stream":
        return run_dual_stream(args)
    args.warmup = max(args.warmup, 3) if args.impl == "product" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    return run_product(args)


if __name__ == "__main__":
    sys.exit(main())
