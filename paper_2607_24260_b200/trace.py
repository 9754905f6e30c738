"""Device-side timeline of the attention kernel, per CTA (a debugging aid, not part of the path).

    python -m paper_2607_24260_b200.trace [c2|c3|c4|c5] [decode|verify] [layers]

Builds the library once more with -DKAP_TRACE (in-tree, `libkap_b200_trace.so`), runs `layers`
consecutive layers of one pass of the named configuration as a CUDA graph and prints, per layer,
when the CTAs entered, finished staging their page ids, passed the dependency wait, saw their
first page, left the main loop and ended - all in microseconds of the GPU's global timer, relative
to the end of the previous layer.  The timestamps themselves cost about 1 us per layer.

Trace slots written by thread 0 of every CTA (see KAP_TRACE_POINT in csrc/kap_attn_kernel.cuh):
0 entry, 1 page ids staged, 2 dependency wait passed, 3 first page arrived, 4 main loop left,
6 warps combined, 5 end; slot 7 holds the SM id.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
TRACE_LIB = os.path.join(HERE, "libkap_b200_trace.so")
RECORDS = 8192                                    # per launch, fixed by the library's trace buffer


def build_trace_library() -> str:
    from . import build
    cmd = [build.NVCC] + build.FLAGS + ["-DKAP_TRACE", "-o", TRACE_LIB] + build.sources()
    subprocess.run(cmd, check=True)
    return TRACE_LIB


def run(config: str = "c2", mode: str = "decode", layers: int = 8):
    from . import build
    build.LIB = build_trace_library()             # before the binding loads the library
    build.is_stale = lambda: False
    import torch
    from . import kap
    sys.path.insert(0, ROOT)
    import bench

    lib = kap.lib()
    cy = bench.Cycle(config, 0, layers=layers)

    def enqueue():
        for layer in range(cy.layers):
            if mode == "decode":
                kap.selected_decode_attn(cy.q_dec[0, layer], cy.pool[layer], cy.d_plan_indptr, cy.d_plan_phys,
                                         cy.d_plan_logical, cy.d_ctx, cy.out_dec[0, layer], cy.ws_d)
            else:
                kap.verify_attn(cy.q_ver[layer], cy.d_q_indptr, cy.pool[layer], cy.d_bt_indptr, cy.d_bt_pages,
                                cy.d_ctx, cy.out_ver[layer], cy.ws_v)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        enqueue()
    stream.synchronize()
    lib.kap_debug_trace_begin.argtypes = [C.c_int]
    lib.kap_debug_trace_read.argtypes = [C.c_void_p, C.c_int]
    if lib.kap_debug_trace_begin(cy.layers) != 0:
        raise RuntimeError("trace buffer allocation failed")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        enqueue()
    for _ in range(5):                            # the last replay's records are the ones read back
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    graph.replay()
    e1.record()
    torch.cuda.synchronize()
    buf = np.zeros((cy.layers, RECORDS, 8), dtype=np.uint64)
    if lib.kap_debug_trace_read(buf.ctypes.data, cy.layers) != 0:
        raise RuntimeError("trace read-back failed")
    info = cy.info_d if mode == "decode" else cy.info_v
    n_ctas = info["n_items"] * info["cluster_size"]
    print(f"{config} {mode}: {e0.elapsed_time(e1) / cy.layers * 1e3:.2f} us per layer with tracing on; schedule {info}")
    report(buf.astype(np.int64), n_ctas, info["cluster_size"])
    return buf


def report(t: np.ndarray, n_ctas: int, cluster: int):
    def stats(a):
        return f"{a.min():6.2f} {np.median(a):6.2f} {a.max():6.2f}"

    print("per layer, us relative to the end of the previous layer (min / median / max over CTAs):")
    for layer in range(1, t.shape[0]):
        r = t[layer, :n_ctas]
        prev_end = t[layer - 1, :n_ctas, 5].max()
        rel = lambda col: (r[:, col] - prev_end) / 1e3
        per_sm = np.bincount(r[:, 7].astype(int), minlength=148)
        clusters = r.reshape(n_ctas // cluster, cluster, 8)
        spread = (clusters[:, :, 4].max(axis=1) - clusters[:, :, 4].min(axis=1)) / 1e3
        tail = (clusters[:, :, 5].max(axis=1) - clusters[:, :, 4].max(axis=1)) / 1e3
        print(f"layer {layer}: entry {stats(rel(0))} | ids staged {stats(rel(1))} | wait passed {stats(rel(2))} | "
              f"first page {stats(rel(3))} | loop left {stats(rel(4))} | end {stats(rel(5))}")
        print(f"         prologue {stats((r[:, 1] - r[:, 0]) / 1e3)} | streaming {stats((r[:, 4] - r[:, 3]) / 1e3)} | "
              f"loop-end spread inside a cluster {stats(spread)} | last loop-end of a cluster to its end {stats(tail)} | "
              f"CTAs per SM histogram {np.bincount(per_sm).tolist()}")


if __name__ == "__main__":
    run(sys.argv[1] if len(sys.argv) > 1 else "c2", sys.argv[2] if len(sys.argv) > 2 else "decode",
        int(sys.argv[3]) if len(sys.argv) > 3 else 8)
