"""Timeline of the decode-attention launches: where the time of a launch goes, CTA by CTA.

Builds the library with -DSAGEKV_TRACE (thread 0 of every CTA of sagekv_decode_attn's kernel notes the global timer
at ten points; the normal build has none of that), replays a CUDA graph of decode calls over the layers of a
workload, and prints the phases of a launch as medians over CTAs and launches.  The stamps cost a few per cent, so
the microseconds per launch printed here are a little above the benchmark's.

    python -m paper_2503_08879_b200.trace [workload] [overlap mode] [layers]
"""

from __future__ import annotations

import ctypes as C
import os
import sys

import numpy as np

NAMES = ["CTA starts", "copies issued", "dependency wait over", "K landed", "maxima exchanged", "weights stored",
         "second product done", "results sent", "inbox full", "CTA ends"]


def main(argv):
    from . import build
    os.environ["SAGEKV_LIB"] = build.build(trace=True)
    import torch
    from . import binding as B, synth
    name = argv[0] if len(argv) > 0 else "C3-2048"
    overlap = int(argv[1]) if len(argv) > 1 else 2
    w = synth.workload(name)
    n_layers = int(argv[2]) if len(argv) > 2 else w.n_layers
    dev = torch.device("cuda:0")
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L, device=dev)
    layers = []
    for l in range(n_layers):
        cache = sk.new_layer(w.n_init, w.n_recent, w.n_sel)
        cache.Kc.normal_(); cache.Vc.normal_()
        cache.state = B.CacheState(w.n_init, w.k_q, w.n_sel, w.n_recent, w.n_recent + 1, w.L, cache.step.data_ptr())
        d = synth.make_decode_inputs(w, l, 0, dev)
        layers.append((cache, d, torch.empty_like(d["q"])))
    sk.set_overlap(overlap)
    steps = 4

    def phase():
        for _ in range(steps):
            for cache, d, out in layers:
                sk.decode_attn(d["q"], d["k_new"], d["v_new"], cache, out)

    phase(); torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        phase()
    for _ in range(3):
        g.replay()
    buf = np.zeros((1 << 15, 12), dtype=np.uint64)
    n = C.c_uint(0)
    B.lib.sagekv_trace_read(buf.ctypes.data_as(C.c_void_p), C.byref(n))           # starts a fresh recording
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (steps * n_layers)
    B.lib.sagekv_trace_read(buf.ctypes.data_as(C.c_void_p), C.byref(n))
    t = buf[: min(n.value, 1 << 15)].astype(np.int64)
    ctas = int(t[0, 11]) * w.n_kv_heads * w.batch
    n_launch = t.shape[0] // ctas
    t = t[np.argsort(t[:, 9])][: n_launch * ctas].reshape(n_launch, ctas, 12)       # launches end one after another
    ends = t[:, :, 9].max(axis=1)
    mid = t[n_launch // 4: n_launch - n_launch // 4]
    prev = ends[n_launch // 4 - 1: n_launch - n_launch // 4 - 1]
    print("%s, overlap mode %d, %d layers: %d CTAs per launch (cluster size %d), %.2f us per launch with the stamps; "
          "launch ends %.0f ns apart (median)" % (name, overlap, n_layers, ctas, int(t[0, 0, 11]), us, np.median(np.diff(ends))))
    print("| phase of a CTA | median ns | 10 % | 90 % |")
    print("|---|---|---|---|")
    for i in range(9):
        d = mid[:, :, i + 1] - mid[:, :, i]
        print("| %s -> %s | %.0f | %.0f | %.0f |" % (NAMES[i], NAMES[i + 1], np.median(d), np.percentile(d, 10), np.percentile(d, 90)))
    print("| previous launch's last CTA ends -> dependency wait over | %.0f | | |" % np.median(mid[:, :, 2] - prev[:, None]))
    print("| CTA starts, relative to the previous launch's end | %.0f | | |" % np.median(mid[:, :, 0] - prev[:, None]))
    print("| CTA ends, relative to its launch's last CTA | %.0f | %.0f | %.0f |" % (
        np.median(mid[:, :, 9] - ends[n_launch // 4: n_launch - n_launch // 4, None]),
        np.percentile(mid[:, :, 9] - ends[n_launch // 4: n_launch - n_launch // 4, None], 10), 0))
    sk.close()


if __name__ == "__main__":
    main(sys.argv[1:])
