#!/usr/bin/env python
"""Benchmark of the SpecPV verification hot path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input:
  refresh step : tree mask -> full verification over the whole cache -> commit of the accepted path
                 (with block-summary update) -> block scores -> selection -> gather into the partial cache
  partial step : tree mask -> partial verification over the partial cache -> commit into its buffer
The cache lengths are put back after every step so that every step sees the same workload.

Prints ONE JSON line (rank 0).  `value` is microseconds per step with all inputs resident in HBM;
`e2e` is the same step through the host-buffer entry point (step tensors copied from pinned host
memory and the outputs copied back inside the timed region); `roofline` is measured live for the
dominant kernel (full-verification attention); `cpu_baseline` times the CPU oracle on a bounded
sample of the same workload.  `--impl reference` times only the oracle.
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
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2512_02337_b200 import workloads as wl  # noqa: E402

METRIC = "verify_attention_us_per_step"
ACCEPT_LEN = 4  # tokens committed per step: the paper's mean accept length is 3.3-3.6 (Table 1), plus the root


# DRAM bytes (read + write) of one full-verification attention launch per layer, from the ncu capture of the
# 2-layer case summarised in profiles/attn_tc_kernel_llama_128k.md; the traffic is proportional to the layers streamed.
NCU_DRAM_BYTES_PER_LAYER = {"llama_128k": (1.075296e9 + 5.433088e6) / 2}


NCU_PARTIAL_DRAM_BYTES_PER_LAYER = (35.098e6 + 0.078e6) / 2  # partial verification at a 4096-token budget, same capture


def ncu_traffic_bytes(workload: str, n_layers: int):
    per_layer = NCU_DRAM_BYTES_PER_LAYER.get(workload)
    return None if per_layer is None else per_layer * n_layers


def load_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t_begin: float = 0.0, t_end: float = float("inf")) -> dict:
        """Summary of the samples that arrived inside [t_begin, t_end] (host clock of the timed region)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for t, r in self.rows:
            if not (t_begin <= t <= t_end + 0.03):
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                power.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(power) if power else None, "reasons": sorted(reasons), "samples": len(sm)}


def build_state(name: str, device, n_layers=None, budget_blocks=None, block_tokens=None):
    """Allocate every buffer of the step once (torch owns device memory; nothing is allocated per step)."""
    from paper_2512_02337_b200 import binding as B
    over = {}
    if block_tokens is not None:  # another page size, the budget kept at the same number of tokens
        base = wl.CONFIGS[name]
        over["bs"] = block_tokens
        over["budget_blocks"] = base["budget_blocks"] * base["bs"] // block_tokens
    if budget_blocks is not None:
        over["budget_blocks"] = budget_blocks
    w = wl.make_workload(name, device=device, n_layers=n_layers, spare_tokens=64, **over)
    c = w.cfg
    L, Hq, Hkv, d, bs, M, batch = c["n_layers"], c["Hq"], c["Hkv"], c["d"], c["bs"], c["M"], w.batch
    sink, local = wl.sink_local_blocks(bs)
    cfg = B.make_config(L, Hq, Hkv, d, bs, c["dtype"], sink, local, c["budget_blocks"], c["buffer_tokens"])
    dt = wl.torch_dtype(c["dtype"])
    max_len = max(c["ctx"]) + 64
    st = dict(w=w, cfg=cfg, B=B, L=L, M=M, batch=batch)
    st["full"] = B.Cache(w.k_pool, w.v_pool, w.block_table, w.seq_lens, max_len)
    st["ws"] = B.new_workspace(cfg, L, batch, max_len, M, device=device)
    st["kmax"] = torch.zeros((L, batch, Hkv, w.max_blocks, d), dtype=dt, device=device)
    st["kmin"] = torch.zeros_like(st["kmax"])
    st["scores"] = torch.zeros((L, batch, Hkv, w.max_blocks), dtype=torch.float32, device=device)
    st["idx"] = torch.zeros((L, batch, Hkv, cfg.budget_blocks), dtype=torch.int32, device=device)
    st["count"] = torch.zeros(batch, dtype=torch.int32, device=device)
    ppb = cfg.budget_blocks + (cfg.buffer_tokens + bs - 1) // bs + 1
    pk = torch.zeros((L, batch * ppb, Hkv, bs, d), dtype=dt, device=device)
    ptable = torch.arange(batch * ppb, dtype=torch.int32, device=device).reshape(batch, ppb).contiguous()
    st["plens"] = torch.zeros(batch, dtype=torch.int32, device=device)
    st["partial"] = B.Cache(pk, torch.zeros_like(pk), ptable, st["plens"], cfg.budget_blocks * bs + cfg.buffer_tokens)
    st["out"] = torch.zeros((L, batch, M, Hq, d), dtype=dt, device=device)
    st["lse"] = torch.zeros((L, batch, M, Hq), dtype=torch.float32, device=device)
    W = (M + 63) // 64
    st["mask_host"] = torch.zeros((batch, M, W), dtype=torch.int64).pin_memory()
    st["mask"] = torch.zeros((batch, M, W), dtype=torch.int64, device=device)
    # accepted path of every sequence: a root-to-node path of ACCEPT_LEN tokens
    acc = np.zeros((batch, 8), dtype=np.int32)
    for b in range(batch):
        depth_of = [len(wl.path_to(w.parents[b], n)) for n in range(M)]
        acc[b, :ACCEPT_LEN] = wl.path_to(w.parents[b], depth_of.index(ACCEPT_LEN))
    st["accepted"] = torch.from_numpy(acc).to(device)
    st["n_accepted"] = torch.full((batch,), ACCEPT_LEN, dtype=torch.int32, device=device)
    st["lens0"] = w.seq_lens.clone()
    st["last_query"] = torch.zeros(batch, dtype=torch.int32, device=device)
    # host copies of the step tensors for the end-to-end path
    st["host"] = {k: getattr(w, k).cpu().pin_memory() for k in ("q", "k_new", "v_new")}
    st["out_host"] = torch.zeros((L, batch, M, Hq, d), dtype=dt).pin_memory()
    st["lse_host"] = torch.zeros((L, batch, M, Hq), dtype=torch.float32).pin_memory()
    # one-time set-up outside the timed region: summaries of the prefilled cache
    B.specpv_update_block_summaries(cfg, 0, L, st["full"], None, w.max_blocks, st["kmax"], st["kmin"], st["ws"])
    torch.cuda.synchronize(device)
    return st


def build_masks(st):
    """a1: tree masks on the host (library routine), then one async copy."""
    B, w = st["B"], st["w"]
    mh = st["mask_host"].numpy().view(np.uint64)
    for b in range(st["batch"]):
        mh[b] = B.specpv_build_tree_mask(w.parents[b], 0, mh.shape[2])
    st["mask"].copy_(st["mask_host"], non_blocking=True)


def run_step(st, e2e: bool, events=None):
    B, w, cfg, L, M, ws = st["B"], st["w"], st["cfg"], st["L"], st["M"], st["ws"]
    full, partial = st["full"], st["partial"]
    # ---- refresh step
    mode = B.specpv_select_mode(int(max(w.cfg["ctx"])), cfg.budget_blocks * cfg.block_tokens, 0, M,
                                cfg.buffer_tokens, 0)
    assert mode == B.MODE_REFRESH
    build_masks(st)
    if events is not None:
        events[0].record()
    if e2e:
        h = st["host"]
        B.specpv_verify_host(cfg, B.MODE_FULL, 0, L, h["q"], h["k_new"], h["v_new"], st["mask_host"], M, full,
                             st["out_host"], st["lse_host"], ws)
    else:
        B.specpv_verify_full(cfg, 0, L, w.q, w.k_new, w.v_new, st["mask"], None, M, full, st["out"], st["lse"], ws)
    if events is not None:
        events[1].record()
    B.specpv_commit_accepted(cfg, 0, L, w.k_new, w.v_new, M, st["accepted"], st["n_accepted"], 8, full,
                             st["kmax"], st["kmin"], ws)
    B.specpv_score_blocks(cfg, 0, L, w.q, None, M, st["last_query"], st["kmax"], st["kmin"], full, st["scores"], ws)
    B.specpv_select_partial_kv(cfg, L, st["scores"], w.seq_lens, st["batch"], w.max_blocks, st["idx"], st["count"], ws)
    B.specpv_refresh_partial(cfg, full, st["idx"], st["count"], partial, st["plens"], ws)
    # ---- partial step
    build_masks(st)
    if events is not None:
        events[2].record()
    if e2e:
        B.specpv_verify_host(cfg, B.MODE_PARTIAL, 0, L, h["q"], h["k_new"], h["v_new"], st["mask_host"], M, partial,
                             st["out_host"], st["lse_host"], ws)
    else:
        B.specpv_verify_partial(cfg, 0, L, w.q, w.k_new, w.v_new, st["mask"], None, M, partial, st["out"],
                                st["lse"], ws)
    if events is not None:
        events[3].record()
    B.specpv_commit_accepted(cfg, 0, L, w.k_new, w.v_new, M, st["accepted"], st["n_accepted"], 8, partial, None,
                             None, ws)
    # put the lengths back so that the next step sees the same workload
    w.seq_lens.copy_(st["lens0"], non_blocking=True)


def timed_loop(st, steps, warmup, e2e, dist_barrier):
    dev = st["w"].device
    for _ in range(warmup):
        run_step(st, e2e)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    dist_barrier()
    launches0 = st["B"].specpv_kernel_launches()
    wall0 = time.time()
    t0.record()
    for i in range(steps):
        run_step(st, e2e, ev[i])
    t1.record()
    torch.cuda.synchronize(dev)
    wall1 = time.time()
    dist_barrier()
    total_ms = t0.elapsed_time(t1)
    full_ms = [e[0].elapsed_time(e[1]) for e in ev]
    part_ms = [e[2].elapsed_time(e[3]) for e in ev]
    st_code, info = st["B"].specpv_poll_status(st["ws"])
    if st_code != 0:
        raise RuntimeError(f"device status {st_code} {info}")
    return total_ms / steps, full_ms, part_ms, st["B"].specpv_kernel_launches() - launches0, (wall0, wall1)


def max_over_ranks(values, device):
    """Every rank's device-timed figures reduced with MAX (replicas run side by side: the job is as slow as
    its slowest rank).  Works on any initialised process group (nccl on GPUs, gloo in the CPU test)."""
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def partial_budget_sweep(st, peaks, budgets=(32, 64, 128), iters=10):
    """Partial verification alone for the partial budgets of the paper's sweep (2048 / 4096 / 8192 tokens at
    64-token blocks): selection and gather with that budget (untimed), then the attention call timed with CUDA
    events.  `frac` is against the HBM time of the bytes that call has to read (partial K/V + step tensors)."""
    B, w, L, M, batch = st["B"], st["w"], st["L"], st["M"], st["batch"]
    c = w.cfg
    bs, Hkv, Hq, d = c["bs"], c["Hkv"], c["Hq"], c["d"]
    dev = w.device
    sink, local = wl.sink_local_blocks(bs)
    out = []
    for budget in budgets:
        cfg = B.make_config(L, Hq, Hkv, d, bs, c["dtype"], sink, local, budget, c["buffer_tokens"])
        idx = torch.zeros((L, batch, Hkv, budget), dtype=torch.int32, device=dev)
        ppb = budget + (cfg.buffer_tokens + bs - 1) // bs + 1
        pk = torch.zeros((L, batch * ppb, Hkv, bs, d), dtype=torch.bfloat16, device=dev)
        plens = torch.zeros(batch, dtype=torch.int32, device=dev)
        ptable = torch.arange(batch * ppb, dtype=torch.int32, device=dev).reshape(batch, ppb).contiguous()
        partial = B.Cache(pk, torch.zeros_like(pk), ptable, plens, budget * bs + cfg.buffer_tokens)
        B.specpv_select_partial_kv(cfg, L, st["scores"], w.seq_lens, batch, w.max_blocks, idx, st["count"], st["ws"])
        B.specpv_refresh_partial(cfg, st["full"], idx, st["count"], partial, plens, st["ws"])
        call = lambda: B.specpv_verify_partial(cfg, 0, L, w.q, w.k_new, w.v_new, st["mask"], None, M, partial,  # noqa: E731
                                               st["out"], st["lse"], st["ws"])
        for _ in range(3):
            call()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        torch.cuda.synchronize(dev)
        for a, b in ev:
            a.record()
            call()
            b.record()
        torch.cuda.synchronize(dev)
        us = statistics.median(a.elapsed_time(b) for a, b in ev) * 1e3
        tokens = int(plens.sum())
        nbytes = L * tokens * Hkv * 2 * d * 2 + L * batch * M * (2 * Hq + 2 * Hkv) * d * 2
        out.append({"budget_tokens": budget * bs, "us": us, "bound_us": nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6,
                    "frac": nbytes / (peaks["hbm_gbs"] * 1e9) / (us * 1e-6), "algorithmic_bytes": nbytes,
                    # DRAM bytes of the partial launch from the 2-layer ncu capture (profiles/attn_tc_kernel_llama_128k.md),
                    # scaled by the layers; only the budget that capture ran at has a figure
                    "traffic": NCU_PARTIAL_DRAM_BYTES_PER_LAYER * L
                    if budget * bs == 4096 and st["w"].name == "llama_128k" and bs == 64 else None})
        del pk, partial
    return out


def per_layer_graph(st, iters=10):
    """The same full and partial verification issued the way a model runs them: one call per layer
    (n_layers = 1), the 32 calls of a pass captured once in a CUDA graph and replayed.  Returns the time of a
    whole pass (all layers) in microseconds for each."""
    B, w, cfg, L, M = st["B"], st["w"], st["cfg"], st["L"], st["M"]
    dev = w.device
    res = {}
    for name, cache in (("full_verify_us", st["full"]), ("partial_verify_us", st["partial"])):
        fn = B.specpv_verify_full if name.startswith("full") else B.specpv_verify_partial
        torch.cuda.synchronize(dev)
        time.sleep(1.0)  # the partial pass is not measured on a device still warm from the full one

        def one_pass():
            for l in range(L):
                fn(cfg, l, 1, w.q[l:l + 1], w.k_new[l:l + 1], w.v_new[l:l + 1], st["mask"], None, M, cache,
                   st["out"][l:l + 1], st["lse"][l:l + 1], st["ws"])
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.stream(side):
            one_pass()  # first calls outside the capture (function attributes are set on first use)
        torch.cuda.current_stream(dev).wait_stream(side)
        torch.cuda.synchronize(dev)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            one_pass()
        for _ in range(3):
            graph.replay()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        torch.cuda.synchronize(dev)
        for a, b in ev:
            a.record()
            graph.replay()
            b.record()
        torch.cuda.synchronize(dev)
        res[name] = statistics.median(a.elapsed_time(b) for a, b in ev) * 1e3
        del graph
    return res


def attention_block(st, peaks, iters=10):
    """The linear maps either side of the attention (QKV projection with rotary embedding, output projection with
    residual) on random-init weights of the model's hidden size: each alone as one layer-batched launch (all
    layers' weights streamed once, more than L2), and the whole block (QKV -> partial verification -> output
    projection) issued per layer and replayed from a CUDA graph.  `frac` is against the HBM time of the weights
    plus the step tensors each launch has to move."""
    B, w, cfg, L, M, batch = st["B"], st["w"], st["cfg"], st["L"], st["M"], st["batch"]
    c = w.cfg
    Hq, Hkv, d = c["Hq"], c["Hkv"], c["d"]
    dev = w.device
    bw = wl.make_block_weights(w.name, device=dev, n_layers=L)
    hid = bw.hidden
    base = (w.seq_lens + 0).to(torch.int32)
    cos_sin = torch.zeros((batch, M, d // 2, 2), dtype=torch.float32, device=dev)
    B.specpv_rope_table(cfg, st["mask"], None, base, batch, M, bw.rope_theta, cos_sin)
    q, k_new, v_new = torch.empty_like(w.q), torch.empty_like(w.k_new), torch.empty_like(w.v_new)
    y = torch.empty_like(bw.x)
    ws = st["ws"]
    es = 2
    calls = {
        "qkv_rope": (lambda: B.specpv_qkv_rope(cfg, 0, L, bw.x, hid, bw.w_qkv, cos_sin, batch, M, q, k_new, v_new, ws),
                     L * ((Hq + 2 * Hkv) * d * hid + batch * M * (hid + (Hq + 2 * Hkv) * d)) * es),
        "o_proj": (lambda: B.specpv_o_proj(cfg, 0, L, st["out"], bw.w_o, hid, bw.residual, batch, M, y, ws),
                   L * (hid * Hq * d + batch * M * (Hq * d + 2 * hid)) * es),
    }
    res = {"hidden": hid}
    for name, (call, nbytes) in calls.items():
        for _ in range(3):
            call()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        torch.cuda.synchronize(dev)
        for a, b in ev:
            a.record()
            call()
            b.record()
        torch.cuda.synchronize(dev)
        us = statistics.median(a.elapsed_time(b) for a, b in ev) * 1e3
        res[name] = {"us": us, "gbs": nbytes / (us * 1e-6) / 1e9, "frac": nbytes / (peaks["hbm_gbs"] * 1e9) / (us * 1e-6)}

    def one_pass():
        for l in range(L):
            B.specpv_qkv_rope(cfg, l, 1, bw.x[l:l + 1], hid, bw.w_qkv, cos_sin, batch, M, q[l:l + 1], k_new[l:l + 1],
                              v_new[l:l + 1], ws)
            B.specpv_verify_partial(cfg, l, 1, q[l:l + 1], k_new[l:l + 1], v_new[l:l + 1], st["mask"], None, M,
                                    st["partial"], st["out"][l:l + 1], st["lse"][l:l + 1], ws)
            B.specpv_o_proj(cfg, l, 1, st["out"][l:l + 1], bw.w_o, hid, bw.residual[l:l + 1], batch, M, y[l:l + 1], ws)
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream(dev))
    with torch.cuda.stream(side):
        one_pass()
    torch.cuda.current_stream(dev).wait_stream(side)
    torch.cuda.synchronize(dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        one_pass()
    for _ in range(3):
        graph.replay()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    torch.cuda.synchronize(dev)
    for a, b in ev:
        a.record()
        graph.replay()
        b.record()
    torch.cuda.synchronize(dev)
    us = statistics.median(a.elapsed_time(b) for a, b in ev) * 1e3
    block_bytes = calls["qkv_rope"][1] + calls["o_proj"][1] + int(st["plens"].sum()) * L * Hkv * 2 * d * es
    res["per_layer_block_graph"] = {"us": us, "bound_us": block_bytes / (peaks["hbm_gbs"] * 1e9) * 1e6,
                                    "frac": block_bytes / (peaks["hbm_gbs"] * 1e9) / (us * 1e-6)}
    del graph
    return res


def offloaded_refresh(st, layers=4, iters=3):
    """The memory-constrained variant (Section 3.3, last paragraph) on the first `layers` layers of the workload: the
    full cache in page-locked host memory, full verification staged through two device layer slots with the next
    layer's copy in flight, and the gather of the selected blocks straight from host memory.  Both are bound by the
    host link, so each is reported with the GB/s it moved over it."""
    B, w, cfg, M, batch = st["B"], st["w"], st["cfg"], st["M"], st["batch"]
    c = w.cfg
    L = min(layers, st["L"])
    Hkv, d, bs = c["Hkv"], c["d"], c["bs"]
    dev = w.device
    dt = wl.torch_dtype(c["dtype"])
    k_host = torch.empty((L,) + tuple(w.k_pool.shape[1:]), dtype=dt).pin_memory()
    v_host = torch.empty_like(k_host).pin_memory()
    k_host.copy_(w.k_pool[:L])
    v_host.copy_(w.v_pool[:L])
    stage_shape = (2,) + tuple(w.k_pool.shape[1:])
    off = B.OffloadedCache(k_host, v_host, torch.zeros(stage_shape, dtype=dt, device=dev),
                           torch.zeros(stage_shape, dtype=dt, device=dev), w.block_table, w.seq_lens, st["full"].max_seq_len)
    cfg_l = B.make_config(L, c["Hq"], Hkv, d, bs, c["dtype"], cfg.sink_blocks, cfg.local_blocks, cfg.budget_blocks,
                          cfg.buffer_tokens)
    copy_stream = torch.cuda.Stream(device=dev)

    def timed(call):
        call()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        torch.cuda.synchronize(dev)
        for a, b in ev:
            a.record()
            call()
            b.record()
        torch.cuda.synchronize(dev)
        return statistics.median(a.elapsed_time(b) for a, b in ev) * 1e3
    layer_bytes = 2 * k_host[0].numel() * k_host.element_size()
    us_v = timed(lambda: B.specpv_verify_full_offloaded(cfg_l, 0, L, w.q[:L], w.k_new[:L], w.v_new[:L], st["mask"], None, M,
                                                        off, st["out"][:L], st["lse"][:L], st["ws"],
                                                        copy_stream=copy_stream))
    # selection for these layers with this budget into buffers of its own (the step's state is left alone)
    idx = torch.zeros((L, batch, Hkv, cfg.budget_blocks), dtype=torch.int32, device=dev)
    count = torch.zeros(batch, dtype=torch.int32, device=dev)
    plens = torch.zeros(batch, dtype=torch.int32, device=dev)
    ppb = cfg.budget_blocks + (cfg.buffer_tokens + bs - 1) // bs + 1
    pk = torch.zeros((L, batch * ppb, Hkv, bs, d), dtype=dt, device=dev)
    ptable = torch.arange(batch * ppb, dtype=torch.int32, device=dev).reshape(batch, ppb).contiguous()
    partial = B.Cache(pk, torch.zeros_like(pk), ptable, plens, cfg.budget_blocks * bs + cfg.buffer_tokens)
    B.specpv_select_partial_kv(cfg_l, L, st["scores"][:L].contiguous(), w.seq_lens, batch, w.max_blocks, idx, count,
                               st["ws"])
    us_g = timed(lambda: B.specpv_refresh_partial(cfg_l, off.as_cache(), idx, count, partial, plens, st["ws"]))
    gathered = L * int(plens.sum()) * Hkv * 2 * d * k_host.element_size()
    res = {"layers": L,
           "full_verify_staged": {"us_per_layer": us_v / L, "h2d_gbs": L * layer_bytes / (us_v * 1e-6) / 1e9,
                                  "bytes_per_layer": layer_bytes},
           "gather_from_host": {"us_per_layer": us_g / L, "host_read_gbs": gathered / (us_g * 1e-6) / 1e9,
                                "bytes_per_layer": gathered // L}}
    del off, k_host, v_host, partial, pk
    return res


def score_variants(st, peaks, iters=10):
    """Block scoring and selection in their variants (Eq. 3's reductions mean / max / last, Eq. 2 as printed and in
    its channel-wise form, selection per head and shared by the heads), each call alone over all layers.  Scoring
    reads the summaries once: `frac` is against the HBM time of those bytes."""
    B, w, L, M, batch = st["B"], st["w"], st["L"], st["M"], st["batch"]
    c = w.cfg
    Hq, Hkv, d, bs = c["Hq"], c["Hkv"], c["d"], c["bs"]
    base = st["cfg"]
    dev = w.device
    nbytes = 2 * st["kmax"].numel() * st["kmax"].element_size() * sum((x + bs - 1) // bs for x in c["ctx"]) \
        // (batch * w.max_blocks)

    def timed(call):
        for _ in range(3):
            call()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        torch.cuda.synchronize(dev)
        for a, b in ev:
            a.record()
            call()
            b.record()
        torch.cuda.synchronize(dev)
        return statistics.median(a.elapsed_time(b) for a, b in ev) * 1e3
    scores = torch.zeros_like(st["scores"])
    idx = torch.zeros_like(st["idx"])
    count = torch.zeros_like(st["count"])
    res = {}
    for label, reduce, mode in (("mean", 0, 0), ("max", 1, 0), ("last", 2, 0), ("mean_channelwise", 0, 1)):
        cfg = B.make_config(L, Hq, Hkv, d, bs, c["dtype"], base.sink_blocks, base.local_blocks, base.budget_blocks,
                            base.buffer_tokens, reduce=reduce, score_mode=mode)
        us = timed(lambda: B.specpv_score_blocks(cfg, 0, L, w.q, None, M, st["last_query"], st["kmax"], st["kmin"],
                                                 st["full"], scores, st["ws"]))
        res["scores_" + label] = {"us": us, "frac": nbytes / (peaks["hbm_gbs"] * 1e9) / (us * 1e-6)}
    for label, shared in (("per_head", 0), ("shared_heads", 1)):
        cfg = B.make_config(L, Hq, Hkv, d, bs, c["dtype"], base.sink_blocks, base.local_blocks, base.budget_blocks,
                            base.buffer_tokens, select_shared=shared)
        us = timed(lambda: B.specpv_select_partial_kv(cfg, L, st["scores"], w.seq_lens, batch, w.max_blocks, idx, count,
                                                      st["ws"]))
        res["select_" + label] = {"us": us}
    return res


def other_workloads(peaks, iters=8):
    """Full verification of the two configurations whose row count differs from the default's, each as one
    layer-batched call timed with CUDA events (median, min) against its own bound (HBM time of the K/V it reads, or
    tensor time of its flops, whichever is longer): the batch-4 ragged stress shape (256 rows per KV head), and a
    refresh step of the 64K decode-loop shape with the partially verified chain in front of the tree (42 + 48 tokens =
    360 rows per KV head: two row groups, the second of which streams the cache again)."""
    from paper_2512_02337_b200 import binding as B
    dev = torch.device("cuda", torch.cuda.current_device())
    res = {}
    for key, name, n_chain, over in (("stress_b4_full_verify", "stress_b4", 0, {}),
                                     ("refresh_chain42_tree48_full_verify", "qwen3_64k_loop", 42, {"M": 90})):
        w = wl.make_workload(name, device=dev, **over)
        c = w.cfg
        L, Hq, Hkv, d, bs, M, batch = c["n_layers"], c["Hq"], c["Hkv"], c["d"], c["bs"], c["M"], w.batch
        sink, local = wl.sink_local_blocks(bs)
        cfg = B.make_config(L, Hq, Hkv, d, bs, c["dtype"], sink, local, c["budget_blocks"], c["buffer_tokens"])
        max_len = max(c["ctx"])
        ws = B.new_workspace(cfg, L, batch, max_len, M, device=dev)
        W = (M + 63) // 64
        mh = np.zeros((batch, M, W), dtype=np.uint64)
        rng = np.random.default_rng(7)
        for b in range(batch):
            parents = wl.make_tree(M - n_chain, 5, 4, rng) if n_chain else w.parents[b]
            mh[b] = B.specpv_build_tree_mask(parents, n_chain, W)
        mask = torch.from_numpy(mh.view(np.int64)).to(dev)
        out = torch.zeros((L, batch, M, Hq, d), dtype=wl.torch_dtype(c["dtype"]), device=dev)
        full = B.Cache(w.k_pool, w.v_pool, w.block_table, w.seq_lens, max_len)
        call = lambda: B.specpv_verify_full(cfg, 0, L, w.q, w.k_new, w.v_new, mask, None, M, full, out, None, ws)  # noqa: E731
        for _ in range(3):
            call()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        torch.cuda.synchronize(dev)
        for a, b in ev:
            a.record()
            call()
            b.record()
        torch.cuda.synchronize(dev)
        code, info = B.specpv_poll_status(ws)
        if code != 0:
            raise RuntimeError(f"device status {code} {info}")
        ts = [a.elapsed_time(b) * 1e3 for a, b in ev]
        tokens = sum(c["ctx"])
        nbytes = L * tokens * Hkv * 2 * d * 2 + L * batch * M * (2 * Hq + 2 * Hkv) * d * 2
        flops = L * Hkv * 4 * (Hq // Hkv) * M * d * (tokens + batch * M)
        t_hbm, t_tensor = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6, flops / (peaks["bf16_tflops"] * 1e12) * 1e6
        us = statistics.median(ts)
        res[key] = {"workload": workload_string(name, c, L, c["budget_blocks"] * bs, batch) + (f", chain {n_chain}" if n_chain else ""),
                    "rows_per_kv_head": (Hq // Hkv) * M, "us_median": us, "us_min": min(ts),
                    "bound": "hbm" if t_hbm >= t_tensor else "tensor", "bound_us": max(t_hbm, t_tensor),
                    "frac": max(t_hbm, t_tensor) / us, "tokens_kv_per_s": L * M * tokens / (us * 1e-6)}
        del w, full, out, ws, call
        torch.cuda.empty_cache()
    return res


def workload_string(name, c, n_layers, budget_tokens, batch):
    """The `config.workload` text, the same in both arms."""
    return (f"{name}: {n_layers} layers, Hq {c['Hq']}, Hkv {c['Hkv']}, d {c['d']}, ctx {c['ctx']}, {c['bs']}-token pages, "
            f"tree {c['M']} nodes, budget {budget_tokens} tokens, batch {batch}")


def algorithmic_work(st):
    """Bytes and flops of one full-verification launch: K/V actually attended + Q, O, Knew, Vnew."""
    c = st["w"].cfg
    es = 2 if c["dtype"] == "bf16" else 4
    L, Hq, Hkv, d, M = st["L"], c["Hq"], c["Hkv"], c["d"], c["M"]
    tokens = sum(c["ctx"])
    kv_bytes = L * tokens * Hkv * 2 * d * es
    step_bytes = L * st["batch"] * M * (2 * Hq + 2 * Hkv) * d * es
    R = (Hq // Hkv) * M
    flops = L * Hkv * 4 * R * d * (tokens + st["batch"] * M)
    return kv_bytes + step_bytes, flops, L * M * tokens


def oracle_sample(st):
    """Time the CPU oracle (as it stands) on one whole layer and scale by the layer count only.

    Sample: layer 0, sequence 0, all KV heads, ALL rows of the step: full verification over the whole context plus
    partial verification over the partial cache; x layers, and for a batch x the sequences' share of the context."""
    import oracle
    w, c = st["w"], st["w"].cfg
    M = c["M"]
    kp, vp = wl.to_numpy(w.k_pool[0]), wl.to_numpy(w.v_pool[0])
    q, kn, vn = (wl.to_numpy(t[0, 0]) for t in (w.q, w.k_new, w.v_new))
    mask = oracle.tree_mask(w.parents[0])
    table = w.block_table[0].cpu().numpy()
    sl = int(st["lens0"][0])
    t0 = time.perf_counter()
    oracle.tree_attention(q, kn, vn, mask, kp, vp, table, sl)
    t_full = time.perf_counter() - t0
    pk, pv = wl.to_numpy(st["partial"].k_pool[0]), wl.to_numpy(st["partial"].v_pool[0])
    plen = st["cfg"].budget_blocks * c["bs"]
    t0 = time.perf_counter()
    oracle.tree_attention(q, kn, vn, mask, pk, pv, st["partial"].block_table[0].cpu().numpy(), plen)
    t_part = time.perf_counter() - t0
    us = (t_full * st["L"] * (sum(c["ctx"]) / c["ctx"][0]) + t_part * st["L"] * st["batch"]) * 1e6
    sample = (f"one whole layer (layer 0, sequence 0, all {c['Hkv']} KV heads, all {M} step tokens): full verify over "
              f"{sl} tokens {t_full:.2f}s + partial verify over {plen} tokens {t_part:.2f}s; x {st['L']} layers"
              + (f" x sequences by context share" if st["batch"] > 1 else "") + "; attention only")
    return us, sample, oracle.num_threads()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama_128k", choices=list(wl.CONFIGS))
    ap.add_argument("--layers", type=int, default=None, help="truncate the layer count (profiling only)")
    ap.add_argument("--budget-blocks", type=int, default=None)
    ap.add_argument("--block-tokens", type=int, default=None, choices=[16, 32, 64],
                    help="tokens per page (default: the workload's 64; the paper's own block size is 16)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the per-layer CUDA-graph measurement")
    ap.add_argument("--no-block", action="store_true",
                    help="skip the QKV / output projection measurement (the linear maps either side of the attention)")
    ap.add_argument("--no-offload", action="store_true",
                    help="skip the host-offloaded full cache measurement (4 layers staged over the host link)")
    ap.add_argument("--no-others", action="store_true", help="skip the stress / refresh-chain full-verification side measurements")
    ap.add_argument("--no-sweep", action="store_true", help="skip the partial-budget sweep (2048/4096/8192 tokens) and the score / selection variants")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        if rank != 0:
            return 0
        return reference_arm(args)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    from paper_2512_02337_b200 import build as build_mod
    if rank == 0 or not (ROOT / "paper_2512_02337_b200" / "lib" / "libspecpv.so").exists():
        build_mod.build()
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        barrier = lambda: dist.barrier()  # noqa: E731
    else:
        barrier = lambda: None  # noqa: E731

    st = build_state(args.workload, dev, args.layers, args.budget_blocks, args.block_tokens)
    c = st["w"].cfg
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else local_rank)
    sampler.start()
    # Generating 17 GB of synthetic caches leaves the device warm and at a power-limited clock for a while: let it settle,
    # so that the warm-up and the timed steps start from the same state on every run (the sampler also delivers its first
    # rows meanwhile).
    torch.cuda.synchronize(dev)
    time.sleep(2.0)
    ms_step, full_ms, part_ms, launches, window = timed_loop(st, args.steps, warmup, False, barrier)
    clocks = sampler.stop(*window)
    e2e = None
    if not args.no_e2e:
        e2e_ms, _, _, _, _ = timed_loop(st, args.steps, warmup, True, barrier)
    if use_dist:
        ms_step, e2e_max = max_over_ranks([ms_step, e2e_ms if not args.no_e2e else 0.0], dev)
        if not args.no_e2e:
            e2e_ms = e2e_max
    # The side measurements below never take the headline line down with them: one that fails (for instance no room for
    # the page-locked host copy of four layers) reports its error text in its place.
    def side(enabled, fn, *fn_args):
        if not (enabled and rank == 0 and c["dtype"] == "bf16"):
            return None
        try:
            # every side measurement starts from a settled device: the section before it leaves the part warm and at a
            # power-limited clock for a while, which moved these figures by up to a third from run to run
            torch.cuda.synchronize(dev)
            time.sleep(1.0)
            return fn(*fn_args)
        except Exception as exc:  # noqa: BLE001
            torch.cuda.synchronize(dev)
            return {"error": f"{type(exc).__name__}: {exc}"[:300]}
    sweep = side(not args.no_sweep and args.budget_blocks is None and args.block_tokens is None, partial_budget_sweep, st,
                 load_peaks())
    graph_times = side(not args.no_graph, per_layer_graph, st)
    block = side(not args.no_block, attention_block, st, load_peaks())
    variants = side(not args.no_sweep, score_variants, st, load_peaks())
    offload = side(not args.no_offload, offloaded_refresh, st)
    others = side(not args.no_others and args.workload == "llama_128k" and args.layers is None, other_workloads, load_peaks())
    if rank != 0:
        return 0

    peaks = load_peaks()
    bytes_full, flops_full, tok_kv = algorithmic_work(st)
    full_avg_s = statistics.mean(full_ms) * 1e-3
    achieved_gbs = bytes_full / full_avg_s / 1e9
    achieved_tf = flops_full / full_avg_s / 1e12
    t_hbm = bytes_full / (peaks["hbm_gbs"] * 1e9)
    t_tensor = flops_full / (peaks["bf16_tflops"] * 1e12)
    bound = "hbm" if t_hbm >= t_tensor or c["dtype"] != "bf16" else "tensor"
    roofline = {"kernel": "full-verification attention (attention + split merge)", "bound": bound,
                "achieved": achieved_gbs if bound == "hbm" else achieved_tf,
                "peak": peaks["hbm_gbs"] if bound == "hbm" else peaks["bf16_tflops"],
                "unit": "GB/s" if bound == "hbm" else "TFLOP/s",
                "frac": (achieved_gbs / peaks["hbm_gbs"]) if bound == "hbm" else achieved_tf / peaks["bf16_tflops"],
                "peak_source": peaks["source"],
                "traffic": ncu_traffic_bytes(args.workload, st["L"]) if args.block_tokens in (None, 64) else None,
                "launch_us": full_avg_s * 1e6, "bound_us": max(t_hbm, t_tensor) * 1e6,
                "achieved_gbs": achieved_gbs, "achieved_tflops": achieved_tf,
                "frac_of_bound": max(t_hbm, t_tensor) / full_avg_s}
    if c["dtype"] == "bf16" and peaks.get("bf16_tflops_sustained"):
        # context: against the GEMM rate measured back to back under the power limit, the flops of this launch need
        # longer than its bytes need at the copy rate, and the kernel runs under that limit too
        roofline["tensor_sustained"] = {"peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                                        "bound_us": flops_full / (peaks["bf16_tflops_sustained"] * 1e12) * 1e6,
                                        "frac": achieved_tf / peaks["bf16_tflops_sustained"]}
    out = {
        "metric": METRIC, "value": ms_step * 1e3, "unit": "us", "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": c["dtype"], "data": "synthetic",
        "config": {"workload": workload_string(args.workload, c, st["L"], st["cfg"].budget_blocks * c["bs"], st["batch"]),
                   "step": "refresh step (full verify + commit + scores + select + gather) + partial step "
                           "(partial verify + commit)",
                   "l2": "inputs larger than L2 (every step streams all layers' caches)",
                   "settle": "2 s idle between building the synthetic caches and the warm-up steps, 1 s before each side measurement",
                   "replicas": "replicas only" if world > 1 else "single GPU"},
        "phases_us": {"full_verify": statistics.mean(full_ms) * 1e3, "partial_verify": statistics.mean(part_ms) * 1e3,
                      "rest": ms_step * 1e3 - statistics.mean(full_ms) * 1e3 - statistics.mean(part_ms) * 1e3},
        "phases_us_median_min": {"full_verify": [statistics.median(full_ms) * 1e3, min(full_ms) * 1e3],
                                 "partial_verify": [statistics.median(part_ms) * 1e3, min(part_ms) * 1e3]},
        "tokens_kv_per_s": world * tok_kv / full_avg_s,
        "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline,
    }
    if not args.no_e2e:
        L, batch, M = st["L"], st["batch"], c["M"]
        es = 2 if c["dtype"] == "bf16" else 4
        h2d = 2 * (L * batch * M * (c["Hq"] + 2 * c["Hkv"]) * c["d"] * es + st["mask_host"].numel() * 8)
        d2h = 2 * (L * batch * M * c["Hq"] * (c["d"] * es + 4))
        out["e2e"] = {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    if sweep is not None:
        out["partial_budget_sweep"] = sweep
    if graph_times is not None:
        out["per_layer_cuda_graph"] = graph_times
    if block is not None:
        out["attention_block"] = block
    if offload is not None:
        out["offloaded_full_cache"] = offload
    if variants is not None:
        out["score_variants"] = variants
    if others is not None:
        out["other_workloads"] = others
    if not args.no_cpu_baseline and world == 1:
        us, sample, cores = oracle_sample(st)
        out["cpu_baseline"] = {"value": us, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample}
    print(json.dumps(out))
    return 0


def reference_arm(args):
    """Times the CPU oracle, as it stands, on the default arm's workload (no GPU work at all).  A step of this arm is
    a bounded sample of the workload's step: one whole layer of sequence 0 (all KV heads, all step tokens, the uncut
    context) through full verification and through partial verification over a cache of the budget's length; the
    value is that time x layers (x the sequences' share of the context for a batch)."""
    import oracle
    name = args.workload
    c = dict(wl.CONFIGS[name])
    n_layers = args.layers or c["n_layers"]
    w = wl.make_workload(name, device="cpu", n_layers=1, ctx=[c["ctx"][0]])
    M = c["M"]
    kp, vp = wl.to_numpy(w.k_pool[0]), wl.to_numpy(w.v_pool[0])
    q, kn, vn = (wl.to_numpy(t[0, 0]) for t in (w.q, w.k_new, w.v_new))
    mask = oracle.tree_mask(w.parents[0])
    table = w.block_table[0].numpy()
    budget = (args.budget_blocks or c["budget_blocks"]) * c["bs"]
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        oracle.tree_attention(q, kn, vn, mask, kp, vp, table, c["ctx"][0])   # full verification, one layer
        oracle.tree_attention(q, kn, vn, mask, kp, vp, table, budget)        # partial verification: a cache of the budget's length
        if i >= args.warmup:
            times.append(time.perf_counter() - t0)
    batch = len(c["ctx"])
    layer_s = statistics.mean(times)
    step_s = layer_s * n_layers * (sum(c["ctx"]) + batch * budget) / (c["ctx"][0] + budget)
    sample = (f"oracle attention of one whole layer per step (sequence 0, all {c['Hkv']} KV heads, all {M} step tokens): full "
              f"verify over {c['ctx'][0]} tokens + partial verify over {budget} tokens, {layer_s:.2f}s; x {n_layers} layers"
              + (" x sequences by context share" if batch > 1 else ""))
    out = {"impl": "reference", "metric": METRIC, "value": step_s * 1e6, "unit": "us", "n_gpus": 1,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": False,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": workload_string(name, c, n_layers, budget, batch)},
           "cpu_baseline": {"value": step_s * 1e6, "unit": "us", "cores": oracle.num_threads(), "kind": "oracle",
                            "sample": sample},
           "e2e": {"value": step_s * 1e6, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
