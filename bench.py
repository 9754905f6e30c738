#!/usr/bin/env python
"""Benchmark of the KAP hot path on B200: plan-guided decode attention tokens/s and HBM GB/s.

A *step* is one propose-k / verify cycle of GraphSpec-style self-speculation (Section 3.2 and the
cost model of Section 4.1, Eq. 7) over one batch, attention only: k selected-KV proposal passes
(every layer: split-K kernel + merge) followed by one full-context verification pass with n_q = k
rows (every layer).  Context length is held constant inside a cycle, as the paper's cost model
assumes.  `value` = B*k proposed tokens per cycle / cycle time, inputs resident in HBM, the whole
cycle replayed as two CUDA graphs (proposal segment, verification segment) with CUDA events
between them.  `e2e` = the same cycle driven from HOST buffers through the C ABI: plan
compilation and scheduling on the host, host->device copies of plan arrays and queries,
device->host copy of every attention output, all inside the timed region (the KV cache itself is
persistent state and stays on the device).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c4] [--no-sweep]
    python bench.py --impl reference ...      # the CPU oracle on the same metric (rank 0 only)
    python bench.py --impl host-plan ...      # host leg only (plan compilation), runs without a GPU

The headline workload is configuration 4 (B = 4, 128K context, all 32 layers, 68.7 GB of KV: the
largest single-GPU configuration, inside the 32K-128K range the target is stated on);
configuration 3 is measured beside it in full, configurations 2 (32 layers), 5 (16 layers) and 1 as
side lines.

N > 1: one process per GPU, every rank runs its own batch (weak scaling, no data-path
collective); time = max over ranks.  Under torchrun the ranks come from the environment; a plain
`python bench.py --gpus N` starts its own N ranks through torch.distributed.run.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "plan-guided decode attn tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def traffic_ratios():
    """dram__bytes_read+write per launch / algorithmic bytes per launch from the last ncu capture
    (profiles/traffic_ratio.txt); None when that capture was taken on other kernel sources"""
    from paper_2607_24260_b200 import traffic
    return traffic.read_ratios()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------- clock sampler
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def __enter__(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.file is None:
            return out
        try:
            self.file.flush()
            with open(self.file.name) as f:
                rows = [r.strip().split(", ") for r in f if r.strip()]
            os.unlink(self.file.name)
        except Exception:
            return out
        sm, reasons = [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0]))
                out["sm_max_mhz"] = float(r[1])
            except ValueError:
                continue
            for name, v in zip(names, r[4:8]):
                if v.strip().lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out["sm_mhz"] = statistics.median(sm)
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# -------------------------------------------------------------------------------- the GPU workload
class Cycle:
    """Device-resident state of one configuration plus the graphs that replay a cycle."""

    def __init__(self, name, seed, layers=None, device="cuda:0", decode_chunk=0, verify_chunk=0,
                 kv_layout="hnd"):
        import torch
        from paper_2607_24260_b200 import kap, synth
        self.torch, self.kap, self.synth = torch, kap, synth
        self.dev = device
        kw = {} if layers is None or name == "c1" else {"layers": layers}
        self.w = w = synth.CONFIGS[name](seed, **kw)
        self.k = int(w.n_q.max())                      # proposal steps per cycle
        self.layers = w.layers
        B, Hq, Hkv, d, P = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size
        self.plan = kap.compile_workload(w)
        self.n_sel = np.diff(self.plan["plan_indptr"])
        self.n_pages = (w.ctx_len.astype(np.int64) + P - 1) // P
        self.decode_bytes = int(self.n_sel.sum()) * w.page_bytes          # per layer, per pass
        self.verify_bytes = int(self.n_pages.sum()) * w.page_bytes
        # KV pool: one slice per layer so that no layer's KV is L2-resident when it is read
        self.pool = torch.empty((self.layers, w.num_pool_pages, 2, Hkv, P, d),
                                dtype=torch.bfloat16, device=device)
        synth.device_fill_normal_(self.pool, 0.5, seed + 1)
        self._plant = name == "c3"      # configuration 3: +2 sigma keys inside the selected pages
        rows_v = int(w.n_q.sum())
        self.q_dec = torch.randn((self.k, self.layers, B, Hq, d), device=device,
                                 generator=self._gen(seed + 2)).to(torch.bfloat16)
        self.q_ver = torch.randn((self.layers, rows_v, Hq, d), device=device,
                                 generator=self._gen(seed + 3)).to(torch.bfloat16)
        self.out_dec = torch.zeros_like(self.q_dec)
        self.out_ver = torch.zeros_like(self.q_ver)
        i32 = lambda a: torch.from_numpy(np.array(a, dtype=np.int32)).to(device)
        if self._plant:
            per_seq = [self.plan["plan_phys_pages"][self.plan["plan_indptr"][b]:self.plan["plan_indptr"][b + 1]]
                       for b in range(B)]
            for layer in range(self.layers):
                synth.plant_affinity_keys_(self.pool[layer], self.q_dec[0, layer], w, per_seq, seed, layer)
        self.d_plan_indptr = i32(self.plan["plan_indptr"])
        self.d_plan_phys = i32(self.plan["plan_phys_pages"])
        self.d_plan_logical = i32(self.plan["plan_logical_pages"])
        self.d_ctx = i32(w.ctx_len)
        self.d_q_indptr = i32(w.q_indptr)
        self.d_bt_indptr = i32(w.bt_indptr)
        self.d_bt_pages = i32(w.bt_pages)
        max_rows = int(w.n_q.max()) * (Hq // Hkv)
        self.ws_d = kap.Workspace(int(device.split(":")[1]), 8192, Hq // Hkv, B)
        self.ws_v = kap.Workspace(int(device.split(":")[1]), 8192, max_rows, B)
        # token-major pools hold the same random values: the attention calls just read them through
        # the other tensor map
        self.pool_attn = self.pool
        if kv_layout == "nhd":
            self.pool_attn = self.pool.view(self.layers, w.num_pool_pages, 2, P, Hkv, d)
            self.ws_d.set_kv_layout(kap.KV_NHD)
            self.ws_v.set_kv_layout(kap.KV_NHD)
        self.info_d = self.ws_d.schedule(self.n_sel, None, Hq, Hkv, decode_chunk)
        self.info_v = self.ws_v.schedule(self.n_pages, w.n_q, Hq, Hkv, verify_chunk)
        self.chunks = (decode_chunk, verify_chunk)
        self.graph_d = self.graph_v = None
        self.launches_per_step = 0

    def _gen(self, seed):
        g = self.torch.Generator(device=self.dev)
        g.manual_seed(seed)
        return g

    # the two segments of a cycle, as plain enqueues (capturable)
    def enqueue_proposal(self):
        kap = self.kap
        for step in range(self.k):
            for layer in range(self.layers):
                kap.selected_decode_attn(self.q_dec[step, layer], self.pool_attn[layer], self.d_plan_indptr,
                                         self.d_plan_phys, self.d_plan_logical, self.d_ctx,
                                         self.out_dec[step, layer], self.ws_d)

    def enqueue_verify(self):
        kap = self.kap
        for layer in range(self.layers):
            kap.verify_attn(self.q_ver[layer], self.d_q_indptr, self.pool_attn[layer], self.d_bt_indptr,
                            self.d_bt_pages, self.d_ctx, self.out_ver[layer], self.ws_v)

    def capture(self):
        torch, kap = self.torch, self.kap
        stream = torch.cuda.Stream(device=self.dev)
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):          # warm-up: tensor maps, function attributes
            self.enqueue_proposal()
            self.enqueue_verify()
        stream.synchronize()
        before = kap.launch_count()
        self.graph_d = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_d, stream=stream):
            self.enqueue_proposal()
        self.graph_v = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_v, stream=stream):
            self.enqueue_verify()
        self.launches_per_step = kap.launch_count() - before
        torch.cuda.synchronize()
        self.ws_d.check()
        self.ws_v.check()

    def time_steps(self, steps, warmup, min_replays=20, min_seconds=0.5):
        """Times EXACTLY `steps` cycles (total and per segment), then goes on replaying until at
        least `min_replays` cycles and `min_seconds` of device time have been timed, for the
        per-step statistics.  Returns (total_ms, decode_ms, verify_ms) of the first `steps` cycles
        and a dict with mean / median / best over all timed cycles."""
        torch = self.torch
        for _ in range(warmup):
            self.graph_d.replay()
            self.graph_v.replay()

        def timed(n):
            ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n)]
            torch.cuda.synchronize()
            for s in range(n):
                ev[s][0].record()
                self.graph_d.replay()
                ev[s][1].record()
                self.graph_v.replay()
                ev[s][2].record()
            torch.cuda.synchronize()
            dec = [e[0].elapsed_time(e[1]) for e in ev]
            ver = [e[1].elapsed_time(e[2]) for e in ev]
            return ev[0][0].elapsed_time(ev[-1][2]), dec, ver

        total, dec, ver = timed(steps)
        all_dec, all_ver = list(dec), list(ver)
        per_step = total / steps
        more = max(min_replays - steps, int(min_seconds * 1e3 / max(per_step, 1e-6)) + 1 - steps, 0)
        if more:
            _, d2, v2 = timed(more)
            all_dec += d2
            all_ver += v2
        cyc = [d + v for d, v in zip(all_dec, all_ver)]
        us_d = lambda ms: ms / (self.k * self.layers) * 1e3
        us_v = lambda ms: ms / self.layers * 1e3
        stats = {"replays": len(cyc), "timed_seconds": round(sum(cyc) * 1e-3, 3),
                 "cycle_ms": {"mean": statistics.fmean(cyc), "median": statistics.median(cyc), "best": min(cyc)},
                 "us_per_layer_decode": {"mean": us_d(statistics.fmean(all_dec)), "median": us_d(statistics.median(all_dec)),
                                         "best": us_d(min(all_dec))},
                 "us_per_layer_verify": {"mean": us_v(statistics.fmean(all_ver)), "median": us_v(statistics.median(all_ver)),
                                         "best": us_v(min(all_ver))}}
        return total, sum(dec), sum(ver), stats

    def free(self):
        for ws in (self.ws_d, self.ws_v):
            ws.close()
        self.graph_d = self.graph_v = None
        self.pool = self.pool_attn = self.q_dec = self.q_ver = self.out_dec = self.out_ver = None
        self.torch.cuda.empty_cache()


def summarise(cy: Cycle, steps, total_ms, dec_ms, ver_ms, n_ranks=1):
    w = cy.w
    peak, peak_kind = measured_peak()
    ms_step = total_ms / steps
    us_dec_layer = dec_ms / steps / (cy.k * cy.layers) * 1e3
    us_ver_layer = ver_ms / steps / cy.layers * 1e3
    gbs_dec = cy.decode_bytes / (us_dec_layer * 1e-6) / 1e9
    gbs_ver = cy.verify_bytes / (us_ver_layer * 1e-6) / 1e9

    ratios = traffic_ratios()

    def roof(kind, gbs, alg_bytes):
        ratio = ratios[kind]
        return {"bound": "hbm", "kernel": f"kap_attn_split_kernel ({kind} launch incl. its merge pass)",
                "achieved": round(gbs, 1), "peak": peak, "unit": "GB/s", "frac": round(gbs / peak, 4),
                "frac_of_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 4), "peak_kind": f"of {peak_kind}",
                "algorithmic_bytes_per_launch": alg_bytes,
                "traffic": None if ratio is None else int(ratio * alg_bytes)}

    return {
        "ms_per_step": ms_step,
        "tokens_per_s": n_ranks * w.batch * cy.k / (ms_step * 1e-3),
        "decode_only_tokens_per_s": n_ranks * w.batch / (dec_ms / steps / cy.k * 1e-3),
        "us_per_layer_decode": round(us_dec_layer, 3),
        "us_per_layer_verify": round(us_ver_layer, 3),
        "decode": roof("decode", gbs_dec, cy.decode_bytes),
        "verify": roof("verify", gbs_ver, cy.verify_bytes),
        "share_decode": dec_ms / (dec_ms + ver_ms),
        "retained_kv_ratio_s": float(cy.n_sel.sum() / cy.n_pages.sum()),
        "schedule": {"decode": cy.info_d, "verify": cy.info_v},
    }


# ------------------------------------------------------------------------------------------- e2e
def time_e2e(cy: Cycle, steps, warmup):
    """The same cycle through the C ABI from HOST buffers: compile + schedule on the host, pinned
    host -> device copies of the plan arrays, context lengths and every query, the two graph
    segments, device -> host copies of every attention output; synchronised per step.  Inside a
    step a second stream carries the copies that the running segment does not need: the
    verification queries go up while the proposal passes run, the proposal outputs come down while
    the verification pass runs."""
    torch, kap, w = cy.torch, cy.kap, cy.w
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype).pin_memory()
    h_q_dec, h_q_ver = pin(cy.q_dec), pin(cy.q_ver)
    h_q_dec.copy_(cy.q_dec)
    h_q_ver.copy_(cy.q_ver)
    h_out_dec, h_out_ver = pin(cy.out_dec), pin(cy.out_ver)
    cap = int(cy.n_pages.sum())
    h_indptr = torch.zeros(w.batch + 1, dtype=torch.int32).pin_memory()
    h_phys = torch.zeros(cap, dtype=torch.int32).pin_memory()
    h_logical = torch.zeros(cap, dtype=torch.int32).pin_memory()
    h_ctx = torch.from_numpy(w.ctx_len.copy()).pin_memory()
    n_plan = int(cy.plan["plan_indptr"][-1])
    h2d = (h_q_dec.numel() + h_q_ver.numel()) * 2 + (h_indptr.numel() + 2 * n_plan + h_ctx.numel()) * 4
    d2h = (h_out_dec.numel() + h_out_ver.numel()) * 2

    side = torch.cuda.Stream(device=cy.dev)
    up_done, qver_done, dec_done = (torch.cuda.Event() for _ in range(3))

    def one_step():
        plan = kap.compile_workload(w)                      # host: Algorithm 1
        n = int(plan["plan_indptr"][-1])
        h_indptr.numpy()[:] = plan["plan_indptr"]
        h_phys.numpy()[:n] = plan["plan_phys_pages"]
        h_logical.numpy()[:n] = plan["plan_logical_pages"]
        cy.ws_d.schedule(np.diff(plan["plan_indptr"]), None, w.num_q_heads, w.num_kv_heads, cy.chunks[0])
        cy.ws_v.schedule(cy.n_pages, w.n_q, w.num_q_heads, w.num_kv_heads, cy.chunks[1])
        cy.d_plan_indptr.copy_(h_indptr, non_blocking=True)
        cy.d_plan_phys[:n].copy_(h_phys[:n], non_blocking=True)
        cy.d_plan_logical[:n].copy_(h_logical[:n], non_blocking=True)
        cy.d_ctx.copy_(h_ctx, non_blocking=True)
        cy.q_dec.copy_(h_q_dec, non_blocking=True)
        main = torch.cuda.current_stream()
        up_done.record(main)
        with torch.cuda.stream(side):
            side.wait_event(up_done)                        # after the proposal queries: same PCIe direction
            cy.q_ver.copy_(h_q_ver, non_blocking=True)
            qver_done.record(side)
        cy.graph_d.replay()
        dec_done.record(main)
        with torch.cuda.stream(side):
            side.wait_event(dec_done)
            h_out_dec.copy_(cy.out_dec, non_blocking=True)
        main.wait_event(qver_done)
        cy.graph_v.replay()
        h_out_ver.copy_(cy.out_ver, non_blocking=True)
        torch.cuda.synchronize()

    for _ in range(warmup):
        one_step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        one_step()
    torch.cuda.synchronize()
    return (time.perf_counter() - t0) * 1e3 / steps, h2d, d2h


# ------------------------------------------------------------------------- the path's other calls
def time_extras(cy: Cycle, vocab: int = 128256, iters: int = 20):
    """Side measurements of the calls around the two attention kernels, on the same workload:
    host plan compilation and scheduling (once per request in the paper), the KV append of one
    token per sequence, Top-3 acceptance over the verification window's logits, and the compact
    view copy the paper's design would make once per request.  Not part of `value`."""
    torch, kap, w = cy.torch, cy.kap, cy.w
    dev = cy.dev
    out = {}
    t0 = time.perf_counter()
    for _ in range(iters):
        plan = kap.compile_workload(w)
    out["compile_plan_ms"] = (time.perf_counter() - t0) / iters * 1e3
    t0 = time.perf_counter()
    for _ in range(iters):        # the host computation itself (kap_schedule skips it when nothing changed)
        kap.schedule_host(cy.n_sel, None, w.num_q_heads, w.num_kv_heads, cy.info_d["ctas_per_wave"],
                          cy.chunks[0], max_cluster=16)
    out["schedule_ms"] = (time.perf_counter() - t0) / iters * 1e3

    def timed(fn):
        """device time per call: `iters` calls captured into one CUDA graph (no host overhead)"""
        stream = torch.cuda.Stream(device=dev)
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):
            fn()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(iters):
                fn()
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters * 1e3          # us

    # append one token per sequence (positions ctx_len-1 rewritten: ctx is not advanced)
    k_new = torch.randn((w.batch, w.num_kv_heads, w.head_dim), device=dev).to(torch.bfloat16)
    ctx_prev = (cy.d_ctx - 1).contiguous()
    out["append_kv_us"] = timed(lambda: kap.append_kv(k_new, k_new, cy.pool[0], cy.d_bt_indptr, cy.d_bt_pages,
                                                       ctx_prev, advance=False))
    # Top-3 acceptance over k + 1 rows per sequence; several logit buffers in turn so that the
    # rows come from HBM, not from L2
    rows = w.batch * (cy.k + 1)
    n_buf = max(2, int(256e6 // (rows * vocab * 4)) + 1)
    logits = [torch.randn((rows, vocab), device=dev, dtype=torch.float32) for _ in range(n_buf)]
    indptr = torch.arange(0, rows + 1, cy.k + 1, device=dev, dtype=torch.int32)
    prop = torch.randint(0, vocab, (rows,), device=dev, dtype=torch.int32)
    top3 = torch.zeros((rows, 3), device=dev, dtype=torch.int32)
    acc = torch.zeros(w.batch, device=dev, dtype=torch.int32)
    nxt = torch.zeros(w.batch, device=dev, dtype=torch.int32)
    turn = [0]

    def accept():
        kap.top3_accept(logits[turn[0] % n_buf], indptr, prop, top3, acc, nxt)
        turn[0] += 1
    us = timed(accept)
    out["top3_accept_us"] = us
    out["top3_accept_GBps"] = rows * vocab * 4 / (us * 1e-6) / 1e9
    out["top3_accept_shape"] = [rows, vocab]
    # compact copy of one layer's selected pages (a different layer each call: no L2 reuse)
    n = int(cy.plan["plan_indptr"][-1])
    compact = torch.empty((3, n) + tuple(cy.pool.shape[2:]), dtype=torch.bfloat16, device=dev)

    def view():
        kap.materialize_view(cy.pool[turn[0] % cy.layers], cy.d_plan_phys, compact[turn[0] % 3])
        turn[0] += 1
    us = timed(view)
    out["materialize_view_us_per_layer"] = us
    out["materialize_view_GBps_read_plus_write"] = 2 * n * w.page_bytes / (us * 1e-6) / 1e9
    # growing plan: compiled once, recent-window entries refreshed on the device every step, the
    # proposal kernel run with token-granular masks (a different layer each call)
    t0 = time.perf_counter()
    for _ in range(iters):
        grow = kap.compile_growing_plan(w.ctx_len, w.span_indptr, w.span_start, w.span_len, w.span_score,
                                        w.budget_tokens, w.n_sink, w.n_recent, w.bt_indptr, w.bt_pages,
                                        force_full=w.force_full, max_growth=4096)
    out["compile_growing_plan_ms"] = (time.perf_counter() - t0) / iters * 1e3
    i32 = lambda a: torch.from_numpy(np.array(a, dtype=np.int32, copy=True)).to(dev)
    g_indptr, g_phys, g_logical = i32(grow["plan_indptr"]), i32(grow["plan_phys_pages"]), i32(grow["plan_logical_pages"])
    g_masks = torch.from_numpy(np.array(grow["plan_token_masks"], copy=True).view(np.int16)).to(dev)
    g_tail = i32(grow["tail_desc"])
    ws = kap.Workspace(int(dev.split(":")[1]), 8192, w.num_q_heads // w.num_kv_heads, w.batch)
    ws.schedule(np.diff(grow["plan_indptr"]), None, w.num_q_heads, w.num_kv_heads)
    out["refresh_recent_us"] = timed(lambda: kap.refresh_recent(
        g_indptr, g_logical, g_phys, g_masks, g_tail, cy.d_bt_indptr, cy.d_bt_pages, cy.d_ctx,
        w.num_pool_pages))
    o = torch.empty_like(cy.q_dec[0, 0])

    def masked():
        layer = turn[0] % cy.layers
        kap.selected_decode_attn(cy.q_dec[0, layer], cy.pool[layer], g_indptr, g_phys, g_logical, cy.d_ctx,
                                 o, ws, plan_token_masks=g_masks)
        turn[0] += 1
    kap.refresh_recent(g_indptr, g_logical, g_phys, g_masks, g_tail, cy.d_bt_indptr, cy.d_bt_pages, cy.d_ctx,
                       w.num_pool_pages)
    torch.cuda.synchronize()
    out["growing_plan_decode_us_per_layer"] = timed(masked)
    ws.check()
    ws.close()
    # full-context decode (the fallback path: identity plan, one query row over the whole block
    # table), the t_full of the paper's cost model
    ws = kap.Workspace(int(dev.split(":")[1]), 8192, w.num_q_heads // w.num_kv_heads, w.batch)
    ws.schedule(cy.n_pages, None, w.num_q_heads, w.num_kv_heads)

    def full():
        layer = turn[0] % cy.layers
        kap.selected_decode_attn(cy.q_dec[0, layer], cy.pool[layer], cy.d_bt_indptr, cy.d_bt_pages, None,
                                 cy.d_ctx, o, ws)
        turn[0] += 1
    out["full_decode_us_per_layer"] = timed(full)
    ws.check()
    ws.close()
    return out


def phase_report(kap, k, t_sel, t_verify, t_full):
    """The paper's phase boundary (Eqs. 6-13) on this run's measured per-layer attention times,
    with the weight terms at zero (attention only): s_time = t_sel / t_full plays the part of the
    retained ratio, the plan pays off iff the acceptance rate h exceeds the break-even value."""
    s_time = t_sel / t_full
    rep = {"k": k, "t_sel_us": t_sel, "t_verify_us": t_verify, "t_full_us": t_full,
           "s_time": s_time,
           # (1 + k h) t_full = k t_sel + t_verify  (Eq. 6 = Eq. 7 with the measured verifier time)
           "break_even_h": max(0.0, (k * t_sel + t_verify - t_full) / (k * t_full))}
    for h in (0.6, 0.8, 1.0):
        m = kap.phase_model(k, h, min(s_time, 1.0), 0.0, 0.0, t_full)
        rep[f"model_speedup_h{h}"] = m["speedup"]                       # verifier at t_full (Eq. 7)
        rep[f"measured_speedup_h{h}"] = (1 + k * h) * t_full / (k * t_sel + t_verify)
    # the fallback controller on the same profiled costs (Section 4.2): what it would decide for a
    # request whose observed Top-3 acceptance is h (1000 verified proposals, attention-only costs)
    verdicts = {}
    for h in (0.02, 0.05, 0.10, 0.50, 0.95):
        d = kap.fallback_decide([int(round(1000 * h))], [1000], [s_time], [t_full], h_min=0.0, s_max=1.0)
        verdicts[f"h={h}"] = {"force_full": int(d["force_full"][0]), "reasons": int(d["reasons"][0]),
                              "slack_us": float(d["slack"][0]), "budget_scale": float(d["budget_scale"][0])}
    rep["fallback_controller"] = verdicts
    return rep


# ---------------------------------------------------------------------------------- CPU baseline
class OracleSampler:
    """Times the oracle, as it stands, on bounded samples of a workload.  A sample unit is one
    sequence of one layer (its proposal-pass attention and its verification attention); the KV
    values of one layer are drawn once on the host (the oracle's time does not depend on them) and
    every unit gets fresh queries.  cycle_seconds() scales the per-sequence times to the whole
    cycle: layers x (k proposal passes + 1 verification pass) over all sequences."""

    def __init__(self, w, seed=0):
        from oracle import kap_oracle as orc
        from paper_2607_24260_b200 import synth
        self.orc, self.synth, self.w = orc, synth, w
        self.plan = orc.compile_workload(w)      # the oracle's own plan: nothing comes from the library
        _, self.pool_bits = synth.host_qkv(w, seed, layer=0, q_rows=1)
        self.t_dec = np.zeros(w.batch)
        self.t_ver = np.zeros(w.batch)
        self.count = np.zeros(w.batch, dtype=np.int64)
        self.units = 0
        self.threads = orc.num_threads()

    def run_units(self, n_units):
        """n_units (sequence, layer) units, sequences taken round-robin; returns seconds spent"""
        w, orc, plan = self.w, self.orc, self.plan
        spent = 0.0
        for _ in range(n_units):
            b = self.units % w.batch
            nq = int(w.n_q[b])
            q = self.synth.normal_bf16((nq, w.num_q_heads, w.head_dim), 1.0,
                                       self.synth.rng_for(self.units, w.name, "oracle-q"))
            lo, hi = int(plan["plan_indptr"][b]), int(plan["plan_indptr"][b + 1])
            t0 = time.perf_counter()
            orc.selected_decode_attn(q[-1:], self.pool_bits, [0, hi - lo], plan["plan_phys_pages"][lo:hi],
                                     plan["plan_logical_pages"][lo:hi], w.ctx_len[b:b + 1])
            t1 = time.perf_counter()
            n_pages = (int(w.ctx_len[b]) + w.page_size - 1) // w.page_size
            orc.verify_attn(q, [0, nq], self.pool_bits, [0, n_pages],
                            w.bt_pages[w.bt_indptr[b]:w.bt_indptr[b] + n_pages], w.ctx_len[b:b + 1])
            t2 = time.perf_counter()
            self.t_dec[b] += t1 - t0
            self.t_ver[b] += t2 - t1
            self.count[b] += 1
            self.units += 1
            spent += t2 - t0
        return spent

    def cycle_seconds(self, k):
        """per-sequence mean times (sequences not sampled yet take the mean of the sampled ones),
        scaled to layers x (k proposal passes + verification) over all sequences"""
        seen = self.count > 0
        dec = np.where(seen, self.t_dec / np.maximum(self.count, 1), 0.0)
        ver = np.where(seen, self.t_ver / np.maximum(self.count, 1), 0.0)
        dec[~seen] = dec[seen].mean()
        ver[~seen] = ver[seen].mean()
        return float(self.w.layers * (k * dec.sum() + ver.sum()))


def cpu_baseline(w, k, budget_s=12.0, min_units=None):
    sm = OracleSampler(w)
    spent = sm.run_units(w.batch if min_units is None else min_units)   # by default every sequence once
    while spent < budget_s and sm.units < w.batch * w.layers:
        spent += sm.run_units(1 if min_units is not None else w.batch)
    cycle_s = sm.cycle_seconds(k)
    return {"value": w.batch * k / cycle_s, "unit": "tokens/s", "cores": sm.threads, "kind": "oracle",
            "sample": f"{sm.units} (sequence, layer) units of {w.name}'s {w.batch * w.layers} (each: proposal-pass "
                      f"attention + verification attention of one sequence in one layer, fp64 C oracle, OpenMP over "
                      f"heads), {spent:.1f} s of CPU work, scaled to a {k}-proposal cycle over {w.layers} layers",
            "s_per_cycle": cycle_s}


# ------------------------------------------------------------------------------------------ main
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), \
        int(os.environ.get("WORLD_SIZE", 1))


def config_dict(w, k, layers, extra=None):
    c = {"workload": f"{w.name}: {w.note}", "batch": w.batch, "ctx_len_max": int(w.ctx_len.max()),
         "ctx_len_min": int(w.ctx_len.min()), "layers": layers, "proposals_per_cycle_k": k,
         "verify_rows": k, "heads": f"{w.num_q_heads}q/{w.num_kv_heads}kv", "head_dim": w.head_dim,
         "page_size": w.page_size}
    kv_bytes = layers * int(sum((int(L) + w.page_size - 1) // w.page_size for L in w.ctx_len)) * w.page_bytes
    c["kv_bytes_per_cycle"] = kv_bytes
    if kv_bytes > 4 * 126e6:
        c["l2"] = "no flush: every layer has its own KV slice, per-cycle working set >> 126 MB L2"
    else:
        c["l2"] = ("small case, no flush: the KV of the whole cycle fits the 126 MB L2, so its figures "
                   "are L2-resident and say nothing about HBM bandwidth")
    if extra:
        c.update(extra)
    return c


def oracle_sample_main(args):
    """--oracle-sample S: time the oracle for about S seconds on the named configuration and print
    the cpu_baseline dict (used by the parent to get a single-thread figure: the child runs with
    OMP_NUM_THREADS=1)."""
    from paper_2607_24260_b200 import synth
    w = synth.CONFIGS[args.config](0)
    print(json.dumps(cpu_baseline(w, int(w.n_q.max()), budget_s=args.oracle_sample, min_units=1)))
    return 0


def cpu_baseline_single_thread(config, budget_s=6.0):
    """the same oracle, one thread: a child process with OMP_NUM_THREADS=1"""
    env = dict(os.environ, OMP_NUM_THREADS="1")
    for key in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        env.pop(key, None)
    try:
        out = subprocess.run([sys.executable, os.path.abspath(__file__), "--config", config,
                              "--oracle-sample", str(budget_s)], env=env, capture_output=True, text=True,
                             timeout=600, check=True).stdout
        return json.loads(out.strip().splitlines()[-1])
    except Exception as e:
        return {"error": repr(e)}


def run_reference(args):
    """--impl reference: the CPU oracle on the same metric and workload (rank 0 only; the other
    ranks exit without work).  Each step times a bounded sample of (sequence, layer) units, sized
    so that warm-up + steps end within about a hundred seconds of oracle work (plus the host-side
    generation of one layer of KV)."""
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    from paper_2607_24260_b200 import synth
    w = synth.CONFIGS[args.config](0)
    k = int(w.n_q.max())
    sm = OracleSampler(w)
    per_step = 100.0 / max(1, args.steps + args.warmup)
    t_unit = sm.run_units(1)                              # calibration
    cycles, units_per_step = [], max(1, int(per_step / max(t_unit, 1e-6)))
    for i in range(args.warmup + args.steps):
        sm.run_units(units_per_step)
        if i >= args.warmup:
            cycles.append(sm.cycle_seconds(k))            # running estimate over everything sampled so far
    ms = cycles[-1] * 1e3
    value = w.batch * k / (ms * 1e-3)
    sample = (f"{units_per_step} (sequence, layer) units per step, {sm.units} sampled in total (the workload has {w.batch * w.layers}; repeats allowed), "
              f"scaled to the full cycle")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s",
            "n_gpus": max(world, args.gpus), "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_dict(w, k, w.layers),
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": sm.threads, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def run_host_plan(args):
    """--impl host-plan: the host leg of the path only - kap_compile_plan on every rank's own batch
    (no GPU work, so it runs anywhere; backend gloo without CUDA).  It exists so that the launch,
    sharding, barrier and max-over-ranks plumbing the GPU arm uses can be run on a CPU machine."""
    import torch
    from paper_2607_24260_b200 import dist as kdist, kap, synth
    rank, local_rank, world = dist_env()
    group = None
    if world > 1:
        cuda = torch.cuda.is_available()
        group = kdist.Group("nccl" if cuda else "gloo", device=f"cuda:{local_rank}" if cuda else "cpu")
    base = synth.CONFIGS[args.config](0, layers=1) if args.config != "c1" else synth.CONFIGS["c1"](0)
    lo, hi = kdist.shard_units(world * base.batch, rank, world)     # this rank's sequences of the global batch
    w = synth.CONFIGS[args.config](lo // base.batch, layers=1) if args.config != "c1" else base
    for _ in range(max(3, args.warmup)):
        kap.compile_workload(w)
    if group:
        group.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        plan = kap.compile_workload(w)
    elapsed = time.perf_counter() - t0
    units = float((hi - lo) * args.steps)
    if group:
        group.barrier()
        value = kdist.aggregate_throughput(units, elapsed, group)
        slowest = group.max_float(elapsed)
    else:
        value, slowest = units / elapsed, elapsed
    if rank == 0:
        print(json.dumps({"impl": "host-plan", "metric": "plans compiled per second (host leg only)", "value": value,
                          "unit": "sequences/s", "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
                          "ms_per_step": slowest / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
                          "config": {"workload": f"{w.name}: {w.note}", "sequences_per_rank": hi - lo,
                                     "pages_selected_rank0": int(plan["plan_indptr"][-1])}}))
    if group:
        group.close()
    return 0


def self_launch(args):
    """`python bench.py --gpus N` without torchrun: start the N ranks ourselves"""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def measure(name, args, dev, seed, group, world, layers=None, want_e2e=True, want_extras=False):
    """One configuration: device-resident cycle timing (exactly args.steps cycles, then the
    per-step statistics), optionally e2e and the side calls.  Returns (result dict, Cycle)."""
    import torch
    if args.lean:
        want_e2e = want_extras = False
    cy = Cycle(name, seed=seed, layers=layers, device=dev, kv_layout=args.kv_layout,
               decode_chunk=args.decode_chunk, verify_chunk=args.verify_chunk)
    cy.capture()
    if group:
        group.barrier()
    torch.cuda.synchronize()
    with ClockSampler(int(dev.split(":")[1])) as clocks:
        total_ms, dec_ms, ver_ms, stats = cy.time_steps(args.steps, max(3, args.warmup),
                                                        *((0, 0.0) if args.lean else ()))
    torch.cuda.synchronize()
    local_ms = total_ms
    if group:
        from paper_2607_24260_b200 import dist as kdist
        group.barrier()
        total_ms = group.max_float(total_ms)
    res = summarise(cy, args.steps, total_ms, dec_ms, ver_ms, n_ranks=world)
    if group:      # all ranks' tokens / the slowest rank's time, through the tested helper
        res["tokens_per_s"] = kdist.aggregate_throughput(float(cy.w.batch * cy.k * args.steps), local_ms * 1e-3, group)
    res["per_step"] = stats
    res["clocks"] = clocks.summary()
    if want_e2e:
        e2e_ms, h2d, d2h = time_e2e(cy, max(3, min(args.steps, 20)), 3)
        if group:
            e2e_ms = group.max_float(e2e_ms)
        res["e2e"] = {"value": world * cy.w.batch * cy.k / (e2e_ms * 1e-3), "unit": "tokens/s",
                      "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                      "note": "per step: host plan compile (Algorithm 1) + both kap_schedule calls (list lengths "
                              "unchanged, so they return without rebuilding: a schedule is per request shape, "
                              "its uncached cost is other_calls.schedule_ms) + H2D of plan arrays, ctx_len and "
                              "every query + the cycle + D2H of every attention output; the KV cache is "
                              "device-resident state"}
    cy.ws_d.check()
    cy.ws_v.check()
    res["gpu_launches"] = cy.launches_per_step * args.steps          # inside the timed region of `value`
    res["per_step"]["gpu_launches_incl_statistics_replays"] = cy.launches_per_step * stats["replays"]
    if want_extras:
        res["other_calls"] = time_extras(cy)
        from paper_2607_24260_b200 import kap
        res["phase"] = phase_report(kap, cy.k, res["us_per_layer_decode"], res["us_per_layer_verify"],
                                    res["other_calls"]["full_decode_us_per_layer"])
    return res, cy


def side_entry(r, cy):
    out = {"workload": cy.w.note, "layers_timed": cy.layers, "replays": r["per_step"]["replays"],
           "timed_seconds": r["per_step"]["timed_seconds"],
           "us_per_layer_decode": r["us_per_layer_decode"], "us_per_layer_verify": r["us_per_layer_verify"],
           "us_per_layer_decode_median_best": [round(r["per_step"]["us_per_layer_decode"][x], 3) for x in ("median", "best")],
           "us_per_layer_verify_median_best": [round(r["per_step"]["us_per_layer_verify"][x], 3) for x in ("median", "best")],
           "decode_GBps": r["decode"]["achieved"], "verify_GBps": r["verify"]["achieved"],
           "decode_frac_of_measured": r["decode"]["frac"], "decode_frac_of_8TBs": r["decode"]["frac_of_nominal_8TBs"],
           "verify_frac_of_measured": r["verify"]["frac"], "verify_frac_of_8TBs": r["verify"]["frac_of_nominal_8TBs"],
           "retained_kv_ratio_s": r["retained_kv_ratio_s"], "decode_only_tokens_per_s": r["decode_only_tokens_per_s"],
           "tokens_per_s": r["tokens_per_s"], "schedule": r["schedule"], "clocks": r["clocks"]}
    for key in ("e2e", "cpu_baseline", "cpu_baseline_single_thread", "roofline_decode", "roofline_verify"):
        if key in r:
            out[key] = r[key]
    return out


class TwoMicroBatches(Cycle):
    """The same configuration run as two micro-batches (first and second half of the sequences) on
    two streams, each an independent chain over the layers - what a serving engine does when it
    interleaves two micro-batches of one forward pass.  The kernels, plans and pool are the same;
    only the launch structure differs: while one chain's launch ramps up, drains or sits at a
    kernel boundary, the other one streams.  A side measurement: it shows what the per-launch
    fixed costs of the single chain cost, it is not the headline."""

    def __init__(self, name, seed, layers=None, device="cuda:0", max_cluster=16, ctas_per_sm=0, restore_max_cluster=16):
        super().__init__(name, seed, layers=layers, device=device)
        torch, kap, w = self.torch, self.kap, self.w
        B, Hq, Hkv = w.batch, w.num_q_heads, w.num_kv_heads
        assert B % 2 == 0
        i32 = lambda a: torch.from_numpy(np.array(a, dtype=np.int32)).to(device)
        self.side = torch.cuda.Stream(device=device)
        self.halves = []
        kap.set_launch_options(-1, -1, ctas_per_sm, max_cluster, -1)     # two launches share the SMs' CTA slots
        try:
            for lo, hi in ((0, B // 2), (B // 2, B)):
                pi, bi = self.plan["plan_indptr"], w.bt_indptr
                h = {"lo": lo, "hi": hi, "rows": (int(w.q_indptr[lo]), int(w.q_indptr[hi])),
                     "plan_indptr": i32(pi[lo:hi + 1] - pi[lo]),
                     "plan_phys": i32(self.plan["plan_phys_pages"][pi[lo]:pi[hi]]),
                     "plan_logical": i32(self.plan["plan_logical_pages"][pi[lo]:pi[hi]]),
                     "ctx": i32(w.ctx_len[lo:hi]), "q_indptr": i32(w.q_indptr[lo:hi + 1] - w.q_indptr[lo]),
                     "bt_indptr": i32(bi[lo:hi + 1] - bi[lo]), "bt_pages": i32(w.bt_pages[bi[lo]:bi[hi]])}
                dev_index = int(device.split(":")[1])
                h["ws_d"] = kap.Workspace(dev_index, 8192, Hq // Hkv, hi - lo)
                h["ws_v"] = kap.Workspace(dev_index, 8192, int(w.n_q.max()) * (Hq // Hkv), hi - lo)
                h["info_d"] = h["ws_d"].schedule(self.n_sel[lo:hi], None, Hq, Hkv)
                h["info_v"] = h["ws_v"].schedule(self.n_pages[lo:hi], w.n_q[lo:hi], Hq, Hkv)
                self.halves.append(h)
        finally:
            kap.set_launch_options(-1, -1, 0, restore_max_cluster, -1)
        self.info_d = [h["info_d"] for h in self.halves]
        self.info_v = [h["info_v"] for h in self.halves]

    def _fork(self, body):
        torch = self.torch
        cur = torch.cuda.current_stream()
        self.side.wait_stream(cur)
        for h, st in zip(self.halves, (cur, self.side)):
            with torch.cuda.stream(st):
                body(h)
        cur.wait_stream(self.side)

    def enqueue_proposal(self):
        kap = self.kap

        def body(h):
            for step in range(self.k):
                for layer in range(self.layers):
                    kap.selected_decode_attn(self.q_dec[step, layer, h["lo"]:h["hi"]], self.pool_attn[layer],
                                             h["plan_indptr"], h["plan_phys"], h["plan_logical"], h["ctx"],
                                             self.out_dec[step, layer, h["lo"]:h["hi"]], h["ws_d"])
        self._fork(body)

    def enqueue_verify(self):
        kap = self.kap

        def body(h):
            r0, r1 = h["rows"]
            for layer in range(self.layers):
                kap.verify_attn(self.q_ver[layer, r0:r1], h["q_indptr"], self.pool_attn[layer], h["bt_indptr"],
                                h["bt_pages"], h["ctx"], self.out_ver[layer, r0:r1], h["ws_v"])
        self._fork(body)

    def free(self):
        for h in self.halves:
            h["ws_d"].check(); h["ws_v"].check()
            h["ws_d"].close(); h["ws_v"].close()
        super().free()


def time_two_microbatches(name, args, dev, layers):
    import torch
    cy = TwoMicroBatches(name, seed=0, layers=layers, device=dev,
                         restore_max_cluster=args.max_cluster if args.max_cluster > 0 else 16)
    cy.capture()
    total_ms, dec_ms, ver_ms, stats = cy.time_steps(args.steps, max(3, args.warmup))
    r = summarise(cy, args.steps, total_ms, dec_ms, ver_ms)
    out = {"workload": cy.w.note, "layers_timed": cy.layers, "replays": stats["replays"],
           "note": "two micro-batches (half of the sequences each) on two streams, each an independent chain of "
                   "layers; same kernels, plans and pool as the headline; per layer = both micro-batches",
           "us_per_layer_decode": r["us_per_layer_decode"], "us_per_layer_verify": r["us_per_layer_verify"],
           "us_per_layer_decode_median_best": [round(stats["us_per_layer_decode"][x], 3) for x in ("median", "best")],
           "us_per_layer_verify_median_best": [round(stats["us_per_layer_verify"][x], 3) for x in ("median", "best")],
           "decode_frac_of_measured": r["decode"]["frac"], "decode_frac_of_8TBs": r["decode"]["frac_of_nominal_8TBs"],
           "verify_frac_of_measured": r["verify"]["frac"], "verify_frac_of_8TBs": r["verify"]["frac_of_nominal_8TBs"],
           "tokens_per_s": r["tokens_per_s"], "schedule": r["schedule"]}
    cy.free()
    return out


def time_c1_warm_cold(args, dev):
    """Configuration 1 (one sequence, one layer, 4096 tokens): its 16.8 MB of KV stay in the L2
    between replays, so one proposal pass and the verification pass are timed twice - replayed
    back to back (warm) and with a 512 MB buffer streamed before every replay (cold: the KV comes
    from HBM again).  Launch-latency bound either way."""
    import torch
    cy = Cycle("c1", seed=0, device=dev, kv_layout=args.kv_layout)
    cy.capture()
    g1 = torch.cuda.CUDAGraph()                       # ONE proposal pass (the cycle's graph holds k)
    stream = torch.cuda.Stream(device=dev)
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g1, stream=stream):
        cy.kap.selected_decode_attn(cy.q_dec[0, 0], cy.pool_attn[0], cy.d_plan_indptr, cy.d_plan_phys,
                                    cy.d_plan_logical, cy.d_ctx, cy.out_dec[0, 0], cy.ws_d)
    flush = torch.zeros(512 << 20, dtype=torch.uint8, device=dev)

    def timed(graph, cold):
        t = []
        for i in range(3 + 20):
            if cold:
                flush.add_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); graph.replay(); e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                t.append(e0.elapsed_time(e1) * 1e3)
        return [round(statistics.median(t), 2), round(min(t), 2)]

    out = {"workload": cy.w.note, "decode_bytes": cy.decode_bytes, "verify_bytes": cy.verify_bytes,
           "note": "one layer, 16.8 MB of KV; [median, best] microseconds over 20 replays; warm = L2-resident, "
                   "cold = 512 MB streamed before every replay; launch-latency bound, not a bandwidth figure"}
    for mode in ("warm", "cold"):
        out[mode] = {"decode_us": timed(g1, mode == "cold"), "verify_us": timed(cy.graph_v, mode == "cold")}

    def chained(enqueue, n=32):
        """Device time per pass when n passes sit in ONE graph (no host launch between them): what
        the pass costs the GPU itself.  The passes read the same L2-resident KV."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(n):
                enqueue()
        t = []
        for i in range(3 + 10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); g.replay(); e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                t.append(e0.elapsed_time(e1) / n * 1e3)
        return [round(statistics.median(t), 2), round(min(t), 2)]

    one_decode = lambda: cy.kap.selected_decode_attn(cy.q_dec[0, 0], cy.pool_attn[0], cy.d_plan_indptr, cy.d_plan_phys,
                                                     cy.d_plan_logical, cy.d_ctx, cy.out_dec[0, 0], cy.ws_d)
    one_verify = lambda: cy.kap.verify_attn(cy.q_ver[0], cy.d_q_indptr, cy.pool_attn[0], cy.d_bt_indptr, cy.d_bt_pages,
                                            cy.d_ctx, cy.out_ver[0], cy.ws_v)
    out["warm_chained"] = {"decode_us": chained(one_decode), "verify_us": chained(one_verify),
                           "note": "32 passes in one graph, per pass: without the host's launch latency"}
    del flush
    cy.free()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "host-plan"])
    ap.add_argument("--config", default="c4", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (debugging)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the other configurations")
    ap.add_argument("--sweep-layers", type=int, default=None, help="layer count of the side configurations")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline legs")
    ap.add_argument("--lean", action="store_true",
                    help="only the --steps timed cycles: no extra replays for the statistics, no e2e, no side "
                         "calls (for runs under a profiler, which should launch as little as possible)")
    ap.add_argument("--oracle-sample", type=float, default=0.0, help=argparse.SUPPRESS)
    ap.add_argument("--max-cluster", type=int, default=-1)
    ap.add_argument("--ring-slots", type=int, default=-1)
    ap.add_argument("--decode-chunk", type=int, default=0, help="cap on pages per CTA, proposal path")
    ap.add_argument("--verify-chunk", type=int, default=0, help="cap on pages per CTA, verification")
    ap.add_argument("--pdl", type=int, default=-1)
    ap.add_argument("--ctas-per-sm", type=int, default=-1)
    ap.add_argument("--early-kv", type=int, default=-1)
    ap.add_argument("--verify-kernel", type=int, default=0, choices=[0, 1],
                    help="kap_set_verify_kernel: 0 = mma.sync split kernel (default), 1 = tcgen05 kernel")
    ap.add_argument("--kv-layout", default="hnd", choices=["hnd", "nhd"],
                    help="pool layout given to the attention calls (default: head-major)")
    args = ap.parse_args()
    if args.oracle_sample > 0:
        return oracle_sample_main(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        return self_launch(args)
    if args.impl == "reference":
        return run_reference(args)
    if args.impl == "host-plan":
        return run_host_plan(args)

    import torch
    from paper_2607_24260_b200 import kap
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    group = None
    if world > 1:
        from paper_2607_24260_b200 import dist as kdist
        group = kdist.Group("nccl", device=dev)
        lo, _ = kdist.shard_units(world * 1, rank, world)    # one batch per rank: weak scaling
        seed = lo
    else:
        seed = 0
    kap.set_launch_options(args.pdl, args.early_kv, args.ctas_per_sm, args.max_cluster, args.ring_slots)
    kap.set_verify_kernel(args.verify_kernel)
    solo = rank == 0 and world == 1

    res, cy = measure(args.config, args, dev, seed, group, world, layers=args.layers, want_extras=solo)
    w, k = cy.w, cy.k
    dominant = "verify" if res["share_decode"] < 0.5 else "decode"
    line = {
        "metric": METRIC, "value": res["tokens_per_s"], "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": res["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": config_dict(w, k, cy.layers, {"parallelism": f"dp{world} (independent batches per GPU)",
                                                 "pdl": args.pdl, "max_cluster": args.max_cluster, "ring_slots": args.ring_slots,
                                                 "ctas_per_sm": args.ctas_per_sm, "early_kv": args.early_kv,
                                                 "kv_layout": args.kv_layout, "verify_kernel": args.verify_kernel}),
        "clocks": res["clocks"], "per_step": res["per_step"], "e2e": res.get("e2e"),
        "gpu_launches": res["gpu_launches"],
        "roofline": res[dominant], "roofline_decode": res["decode"], "roofline_verify": res["verify"],
        "us_per_layer_decode": res["us_per_layer_decode"],
        "us_per_layer_verify": res["us_per_layer_verify"],
        "decode_only_tokens_per_s": res["decode_only_tokens_per_s"],
        "retained_kv_ratio_s": res["retained_kv_ratio_s"], "schedule": res["schedule"],
    }
    for key in ("other_calls", "phase"):
        if key in res:
            line[key] = res[key]
    cy.free()

    if solo and not args.no_sweep and not args.lean:
        also = {}
        plan = [n for n in ("c4", "c3", "c2", "c5") if n != args.config]
        for name in plan:
            try:
                full = name in ("c3", "c4")                  # measured like the headline: e2e and CPU baseline too
                layers = args.sweep_layers if args.sweep_layers else None    # each at its own full layer count
                r, c2 = measure(name, args, dev, 0, None, 1, layers=layers, want_e2e=full)
                if full and not args.no_cpu:          # all cores; the one-thread figure is the headline's only
                    r["cpu_baseline"] = cpu_baseline(c2.w, c2.k)
                if full:
                    r["roofline_decode"], r["roofline_verify"] = r["decode"], r["verify"]
                also[name] = side_entry(r, c2)
                c2.free()
            except Exception as e:       # a side measurement must not lose the main line
                also[name] = {"error": repr(e)}
        try:       # verification through the tcgen05 kernel (8 layers each), for the record: it is the slower one
            kap.set_verify_kernel(1)
            tc = {}
            for name in ("c4", "c3"):
                c3 = Cycle(name, 0, layers=8, device=dev, kv_layout=args.kv_layout)
                c3.capture()
                _, _, _, st = c3.time_steps(3, 3, min_replays=20, min_seconds=0.3)
                tc[name] = {"us_per_layer_verify_mean_median_best": [round(st["us_per_layer_verify"][q], 2) for q in ("mean", "median", "best")],
                            "verify_frac_of_8TBs": round(c3.verify_bytes / (st["us_per_layer_verify"]["mean"] * 1e-6) / 8e12, 4),
                            "schedule": c3.info_v}
                c3.free()
            tc["note"] = "kap_set_verify_kernel(1): tcgen05.mma, accumulators in tensor memory; 8 layers"
            also["verify_tcgen05"] = tc
        except Exception as e:
            also["verify_tcgen05"] = {"error": repr(e)}
        finally:
            kap.set_verify_kernel(args.verify_kernel)
        try:       # the headline configuration once more, as two interleaved micro-batches (8 layers)
            also[args.config + "_two_microbatches"] = time_two_microbatches(args.config, args, dev, 8)
        except Exception as e:
            also[args.config + "_two_microbatches"] = {"error": repr(e)}
        try:
            also["c1"] = time_c1_warm_cold(args, dev)
        except Exception as e:
            also["c1"] = {"error": repr(e)}
        line["also"] = also
    if solo and not args.no_cpu and not args.lean:
        line["cpu_baseline"] = cpu_baseline(w, k)
        line["cpu_baseline_single_thread"] = cpu_baseline_single_thread(args.config)
    if rank == 0:
        print(json.dumps(line))
    if group:
        group.close()
    return 0


if __name__ == "__main__":
    sys.exit(main())
