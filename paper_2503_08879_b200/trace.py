"""Timeline of the decode-attention (or select+compact) launches: where the time of a launch goes, CTA by CTA.

Builds the library with -DSAGEKV_TRACE (thread 0 of every CTA of the kernel notes the global timer at ten points;
the normal build has none of that), replays a CUDA graph of decode calls (select calls in hint mode 2 with
`--select`) over the layers of a workload, and prints the phases of a launch as medians over CTAs and launches.
The stamps cost a few per cent, so the microseconds per launch printed here are a little above the benchmark's.

    python -m paper_2503_08879_b200.trace [workload] [overlap mode] [layers] [decode variant] [--select]
"""

from __future__ import annotations

import ctypes as C
import os
import sys

import numpy as np

# (in select overlap mode 2 the dependency wait sits between "slots written" and "rows moved", not at the entry)
SELECT_NAMES = ["CTA starts", "entry done", "candidate list in shared memory", "cut bin found",
                "candidates flagged", "border ranked", "slots written", "rows moved", "step word", "CTA ends"]
NAMES = ["CTA starts", "copies issued", "dependency wait over", "K landed", "maxima exchanged", "weights stored",
         "second product done", "results sent", "inbox full", "CTA ends"]


def report(buf_reader, names, ctas_of, run, label):
    """Records one run and prints the phases; ctas_of(first record) = CTAs per launch."""
    import torch
    buf = np.zeros((1 << 15, 12), dtype=np.uint64)
    n = C.c_uint(0)
    buf_reader(buf.ctypes.data_as(C.c_void_p), C.byref(n))                         # starts a fresh recording
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); n_calls = run(); e1.record(); torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n_calls
    buf_reader(buf.ctypes.data_as(C.c_void_p), C.byref(n))
    t = buf[: min(n.value, 1 << 15)].astype(np.int64)
    grid = t[:, 11] & 0xffffffff
    tags = t[:, 11] >> 32                          # which buffer the launch wrote: one value per layer
    ctas = ctas_of(np.concatenate([t[0, :11], grid[:1]]))
    groups = []                                    # launches may overlap in time: told apart by tag, then by start
    for tag in np.unique(tags):
        r = t[tags == tag]
        r = r[np.argsort(r[:, 0])]
        for k in range(r.shape[0] // ctas):
            groups.append(r[k * ctas: (k + 1) * ctas])
    groups.sort(key=lambda g_: g_[:, 9].max())
    t = np.stack(groups)
    n_launch = t.shape[0]
    ends = t[:, :, 9].max(axis=1)
    lo, hi = n_launch // 4, n_launch - n_launch // 4
    mid, prev = t[lo:hi], ends[lo - 1: hi - 1]
    print("%s: %d CTAs per launch, %.2f us per launch with the stamps; launch ends %.0f ns apart (median)" % (
        label, ctas, us, np.median(np.diff(ends))))
    print("| phase of a CTA | median ns | 10 % | 90 % |")
    print("|---|---|---|---|")
    for i in range(9):
        d = mid[:, :, i + 1] - mid[:, :, i]
        print("| %s -> %s | %.0f | %.0f | %.0f |" % (names[i], names[i + 1], np.median(d), np.percentile(d, 10), np.percentile(d, 90)))
    if "dependency wait over" in names:
        print("| previous launch's last CTA ends -> dependency wait over | %.0f | | |" % np.median(mid[:, :, names.index("dependency wait over")] - prev[:, None]))
    print("| CTA starts, relative to the previous launch's end | %.0f | | |" % np.median(mid[:, :, 0] - prev[:, None]))
    rel = mid[:, :, 9] - ends[lo:hi, None]
    print("| CTA ends, relative to its launch's last CTA | %.0f | %.0f | %.0f |" % (np.median(rel), np.percentile(rel, 10), 0))


def trace_select(argv):
    """Select+compact launches in hint mode 2 over the layers of a workload (scores and lists from sagekv_score)."""
    import torch
    from . import binding as B, synth
    name = argv[0] if len(argv) > 0 else "C3-2048"
    overlap = int(argv[1]) if len(argv) > 1 else 2
    w = synth.workload(name)
    n_layers = int(argv[2]) if len(argv) > 2 else min(16, w.n_layers)
    dev = torch.device("cuda:0")
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L, device=dev)
    sk.set_select_hint(2, w.n_sel)
    stride = sk.score_stride(w.n_ctx, w.n_init, w.n_recent)
    layers = []
    for l in range(n_layers):
        lay = synth.make_layer(w, l, dev)
        lay["scores"] = torch.empty(w.batch * w.n_q_heads, stride, dtype=torch.float32, device=dev)
        lay["cache"] = sk.new_layer(w.n_init, w.n_recent, w.n_sel)
        B.sagekv_score(sk.ctx, lay["q_last"], lay["K"], w.n_ctx, w.n_init, w.n_recent, lay["scores"], stride)
        layers.append(lay)
    sk.set_select_overlap(overlap)
    rounds = 4

    def phase():
        for _ in range(rounds):
            for lay in layers:
                c = lay["cache"]
                B.sagekv_select_compact(sk.ctx, lay["scores"], stride, lay["K"], lay["V"], w.n_ctx, w.n_init, w.n_recent,
                                        w.n_sel, c.idx, c.Kc, c.Vc, c.state)

    phase(); torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        phase()
    for _ in range(3):
        g.replay()

    def run():
        g.replay()
        return rounds * n_layers

    report(B.lib.sagekv_trace_read_select, SELECT_NAMES, lambda r: int(r[11]), run,
           "%s select+compact, hint mode 2, overlap mode %d, %d layers" % (name, overlap, n_layers))
    sk.close()


def main(argv):
    from . import build
    os.environ["SAGEKV_LIB"] = build.build(trace=True)
    import torch
    from . import binding as B, synth
    if "--select" in argv:
        return trace_select([a for a in argv if a != "--select"])
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
    sk.set_decode_variant(int(argv[3]) if len(argv) > 3 else 0)
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

    def run():
        g.replay()
        return steps * n_layers

    report(B.lib.sagekv_trace_read, NAMES, lambda r: int(r[11]) * w.n_kv_heads * w.batch, run,
           "%s decode, overlap mode %d, %d layers (cluster size %s)" % (name, overlap, n_layers, "= CTAs / (KV heads x batch)"))
    sk.close()


if __name__ == "__main__":
    main(sys.argv[1:])
