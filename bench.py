#!/usr/bin/env python
"""Benchmark of the SAGE-KV hot path on synthetic Llama-3.1-8B-shaped caches at 128K context.

One step = one pass of the whole path over the 32-layer stack of the workload:
  phase A  sagekv_score           once per layer   (last-token query over the eviction region)
  phase B  sagekv_select_compact  once per layer   (top-k per query head + gather of the reduced cache)
  phase C  sagekv_decode_attn     decode_steps x layers (append to the recent window + split-K attention)
Each phase is captured once in a CUDA graph and replayed, so the timed region contains kernel work
rather than Python launch overhead.  Inputs are generated on the GPU before the timed region.  The
layers are visited round-robin and every phase touches more bytes than the L2 holds between two
visits of the same buffer (K alone is 268 MB per layer), so no separate L2 flush is needed.

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle instead.
"""

from __future__ import annotations

import argparse
import hashlib
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

METRIC = "sagekv_select_compact_us_per_layer_128k"
UNIT = "us/layer"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(w):
    """Bytes each call has to move per layer (scores re-read from L2 in later radix passes not counted)."""
    B, Hq, Hkv, d, E, L, K = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.E, w.L, w.n_sel
    score = B * (Hkv * E * d * 2 + Hq * E * 4)
    select = B * (Hq * E * 4 + 2 * (Hkv * L * d * 2 * 2) + Hkv * K * 4)
    decode = B * (Hkv * L * d * 2 * 2)
    return {"score": score, "select_compact": select, "decode_attn": decode}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.thread = [], None, None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        if self.thread:
            self.thread.join(timeout=2)
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def source_hash(files) -> str:
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2503_08879_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str, files):
    """DRAM bytes per launch from the committed ncu summary, or None if the kernel's source changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            rec = json.load(f)[kernel]
        return rec["dram_bytes_per_launch"] if rec.get("source_hash") == source_hash(files) else None
    except Exception:
        return None


# ------------------------------------------------------------------------------------------- oracle arm

def time_oracle_layer(w, lay_cpu, n_decode=1):
    """Wall-clock seconds of the CPU oracle on one layer: score, select+compact, one decode step."""
    import numpy as np
    import torch
    from oracle import sagekv_oracle as O
    from paper_2503_08879_b200 import synth
    bits = lambda t: t.contiguous().view(torch.uint16).numpy()
    q, K, V = bits(lay_cpu["q_last"][0]), bits(lay_cpu["K"][0]), bits(lay_cpu["V"][0])
    t0 = time.perf_counter()
    p = O.score(q, K, w.n_init, w.n_recent).astype(np.float32)
    t1 = time.perf_counter()
    idx = O.select(p, w.k_q, w.n_init)
    Kc, Vc = O.compact(K, V, idx, w.n_init, w.n_recent)
    t2 = time.perf_counter()
    d = synth.make_decode_inputs(w, 0, 0, "cpu")
    for _ in range(n_decode):
        O.decode_step(bits(d["q"][0]), bits(d["k_new"][0]), bits(d["v_new"][0]), Kc, Vc, 0, w.n_init, w.k_q, w.n_recent)
    t3 = time.perf_counter()
    return {"score_s": t1 - t0, "select_compact_s": t2 - t1, "decode_step_s": (t3 - t2) / n_decode}


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return 1


def run_reference(args, w):
    """The oracle as it stands, on the host cores: each step is one layer of the workload."""
    import torch
    from paper_2503_08879_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    torch.manual_seed(0)
    lay = synth.make_layer(w.with_(batch=1), 0, "cpu")
    for _ in range(args.warmup):
        time_oracle_layer(w, lay)
    times = [time_oracle_layer(w, lay) for _ in range(args.steps)]
    sel_us = statistics.mean(t["select_compact_s"] for t in times) * 1e6
    total_ms = statistics.mean(sum(t.values()) for t in times) * 1e3
    cores = os.cpu_count()
    line = {
        "impl": "reference", "metric": METRIC, "value": sel_us, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "n_ctx": w.n_ctx, "budget": w.budget, "layers_per_step": 1},
        "cpu_baseline": {"value": sel_us, "unit": UNIT, "cores": 1, "kind": "oracle", "host_cores": cores,
                         "sample": "1 layer of %s per step: numpy select (lexsort) + row-copy compact, single thread; "
                                   "score %.2f s/layer on %d BLAS threads and decode %.1f ms/layer-step timed beside it"
                                   % (w.name, statistics.mean(t["score_s"] for t in times), blas_threads(),
                                      statistics.mean(t["decode_step_s"] for t in times) * 1e3)},
        "e2e": {"value": sel_us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------- CUDA arm

class Stack:
    """The layers of one workload resident on the device, and CUDA graphs of the three phases over them."""

    def __init__(self, B, synth, torch, w, n_layers, graph_steps, dev, hint):
        self.B, self.torch, self.w, self.dev = B, torch, w, dev
        self.n_layers, self.graph_steps = n_layers, graph_steps
        self.sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L, device=dev)
        strides = []
        for mode in (0, 1, 2):                      # one score buffer serves every hint mode: the widest stride
            self.sk.set_select_hint(mode, w.n_sel)
            strides.append(self.sk.score_stride(w.n_ctx, w.n_init, w.n_recent))
        self.stride = max(strides)
        self.set_hint(hint)
        self.layers = []
        for l in range(n_layers):
            lay = synth.make_layer(w, l, dev)
            lay.pop("heavy")
            lay["scores"] = torch.empty(w.batch * w.n_q_heads, self.stride, dtype=torch.float32, device=dev)
            lay["cache"] = self.sk.new_layer(w.n_init, w.n_recent, w.n_sel)
            lay["out"] = torch.empty(w.batch, w.n_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
            lay["dec"] = [synth.make_decode_inputs(w, l, t, dev) for t in range(graph_steps)]
            self.layers.append(lay)
        torch.cuda.synchronize()

    def set_hint(self, mode):
        self.hint = mode
        self.sk.set_select_hint(mode, self.w.n_sel)

    def phase_a(self):
        w = self.w
        for lay in self.layers:
            self.B.sagekv_score(self.sk.ctx, lay["q_last"], lay["K"], w.n_ctx, w.n_init, w.n_recent, lay["scores"], self.stride)

    def phase_b(self):
        w = self.w
        for lay in self.layers:
            c = lay["cache"]
            self.B.sagekv_select_compact(self.sk.ctx, lay["scores"], self.stride, lay["K"], lay["V"], w.n_ctx, w.n_init,
                                         w.n_recent, w.n_sel, c.idx, c.Kc, c.Vc, c.state)

    def phase_c(self):
        for t in range(self.graph_steps):
            for lay in self.layers:
                d = lay["dec"][t]
                self.sk.decode_attn(d["q"], d["k_new"], d["v_new"], lay["cache"], lay["out"])

    def graph(self, fn):
        fn()                                         # eager once: loads modules, sets function attributes
        self.torch.cuda.synchronize()
        g = self.torch.cuda.CUDAGraph()
        with self.torch.cuda.graph(g):
            fn()
        return g

    def time_graph(self, g, replays, reps):
        """Mean milliseconds of `replays` back-to-back replays, over `reps` measurements after one warm-up."""
        torch = self.torch
        for _ in range(replays):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        tot = 0.0
        for _ in range(reps):
            e0.record()
            for _ in range(replays):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            tot += e0.elapsed_time(e1)
        return tot / reps

    def check(self, O):
        """Layer 0 of what was timed against the oracle: scores, indices, reduced cache, one decode step."""
        import numpy as np
        torch, w, lay = self.torch, self.w, self.layers[0]
        bits = lambda t: t.detach().cpu().contiguous().view(torch.uint16).numpy()
        self.phase_a(); self.phase_b()
        torch.cuda.synchronize()
        cache = lay["cache"]
        ok = True
        refs = []
        for b in range(w.batch):
            got = lay["scores"].view(w.batch, w.n_q_heads, -1)[b, :, : w.E].cpu().numpy()
            ref = O.score(bits(lay["q_last"][b]), bits(lay["K"][b]), w.n_init, w.n_recent)
            ok &= bool(np.all(np.abs(got - ref) <= 1e-3 * np.abs(ref) + 1e-30))
            idx = cache.indices()[b].cpu().numpy()
            ok &= bool(np.array_equal(idx, O.select(got, w.k_q, w.n_init)))
            Kc_ref, Vc_ref = O.compact(bits(lay["K"][b]), bits(lay["V"][b]), idx, w.n_init, w.n_recent)
            Kc, Vc = cache.cache()
            ok &= bool(np.array_equal(bits(Kc[b]), Kc_ref) and np.array_equal(bits(Vc[b]), Vc_ref))
            refs.append((Kc_ref, Vc_ref))
        d = lay["dec"][0]
        out = self.sk.decode_attn(d["q"], d["k_new"], d["v_new"], cache)      # one step with append, step counter 0
        torch.cuda.synchronize()
        for b in range(w.batch):
            o_ref, _, _ = O.decode_step(bits(d["q"][b]), bits(d["k_new"][b]), bits(d["v_new"][b]), refs[b][0], refs[b][1], 0,
                                        w.n_init, w.k_q, w.n_recent)
            ok &= bool(np.all(np.abs(out[b].float().cpu().numpy() - o_ref) <= 1e-2 + 1e-2 * np.abs(o_ref)))
        return ok

    def close(self):
        self.sk.close()
        self.layers = []


def side_workload(B, synth, torch, name, n_layers, dev, hint, check, O):
    """select+compact, score and decode per layer on a few layers of another workload (not part of the timed step)."""
    w = synth.workload(name)
    st = Stack(B, synth, torch, w, n_layers, 4, dev, hint)
    st.sk.set_overlap(2)
    st.sk.set_select_overlap(2)
    ga, gb, gc = st.graph(st.phase_a), st.graph(st.phase_b), st.graph(st.phase_c)
    a = st.time_graph(ga, 2, 3) * 1e3 / (2 * n_layers)
    b = st.time_graph(gb, 2, 3) * 1e3 / (2 * n_layers)
    c = st.time_graph(gc, 8, 3) * 1e3 / (8 * 4 * n_layers)
    ab = algorithmic_bytes(w)
    peak, _ = measured_peak()
    rec = {"workload": name, "layers_timed": n_layers, "of_layers": w.n_layers, "batch": w.batch, "select_hint_mode": hint,
           "score_us_per_layer": a, "select_compact_us_per_layer": b, "decode_attn_us_per_layer_step": c,
           "frac_of_peak": {"score": ab["score"] / (a * 1e-6) / 1e9 / peak,
                            "select_compact": ab["select_compact"] / (b * 1e-6) / 1e9 / peak,
                            "decode_attn": ab["decode_attn"] / (c * 1e-6) / 1e9 / peak}}
    if check:
        rec["parity"] = st.check(O)
    st.close()
    del st
    torch.cuda.empty_cache()
    return rec


def run_cuda(args, w):
    import torch
    from paper_2503_08879_b200 import build as _build, replicas, synth
    rank, local_rank, world = replicas.env_world()
    if world != args.gpus and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    if rank == 0:
        _build.build()
    replicas.init("nccl", dev)
    replicas.barrier()
    from paper_2503_08879_b200 import binding as B
    O = None
    if args.check:
        from oracle import sagekv_oracle as O

    n_layers = args.layers or w.n_layers
    decode_steps = args.decode_steps if args.decode_steps is not None else w.decode_steps
    graph_steps = min(8, max(1, decode_steps))
    decode_steps = (decode_steps // graph_steps) * graph_steps
    hint = args.hint
    st = Stack(B, synth, torch, w, n_layers, graph_steps, dev, hint)
    sk, layers = st.sk, st.layers

    # decode launches overlap with their predecessor; with several layers the kernel before a decode call
    # belongs to another layer, so the reduced cache may be fetched before the dependency wait
    overlap = args.overlap if args.overlap is not None else (2 if n_layers > 1 else 1)
    sk.set_overlap(overlap)
    sk.set_decode_variant(args.decode_variant)
    # the select calls of the layers are queued one after another (phase B follows the score calls of every layer),
    # so no select launch's predecessor writes its inputs: the selection may run ahead of the dependency wait
    sel_overlap = args.select_overlap if args.select_overlap is not None else (2 if n_layers > 1 else 1)
    sk.set_select_overlap(sel_overlap)
    ga, gb, gc = st.graph(st.phase_a), st.graph(st.phase_b), st.graph(st.phase_c)
    c_replays = decode_steps // graph_steps

    def step(ev=None):
        if ev: ev[0].record()
        ga.replay()
        if ev: ev[1].record()
        gb.replay()
        if ev: ev[2].record()
        for _ in range(c_replays):
            gc.replay()
        if ev: ev[3].record()

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    replicas.barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    torch.cuda.synchronize()
    t_wall0 = time.perf_counter()
    for s_ in range(args.steps):
        step(evs[s_])
    torch.cuda.synchronize()
    t_wall = time.perf_counter() - t_wall0
    replicas.barrier()
    clocks = sampler.stop() if rank == 0 else None

    ms = lambda a, b: a.elapsed_time(b)
    tot_ms = sum(ms(e[0], e[3]) for e in evs) / args.steps
    a_us = sum(ms(e[0], e[1]) for e in evs) / args.steps * 1e3 / n_layers
    b_us = sum(ms(e[1], e[2]) for e in evs) / args.steps * 1e3 / n_layers
    c_launches = decode_steps * n_layers
    c_us = (sum(ms(e[2], e[3]) for e in evs) / args.steps * 1e3 / c_launches) if c_launches else float("nan")
    tot_ms = replicas.max_over_ranks(tot_ms, dev)
    a_us, b_us, c_us = (replicas.max_over_ranks(x, dev) for x in (a_us, b_us, c_us))

    # ---- beside the timed step (rank 0, one GPU): the other settings of the same calls, and the Qwen shape ----
    by_hint, by_overlap, by_sel_overlap, by_variant, other, parity = {}, {}, {}, {}, [], None
    if rank == 0 and args.gpus == 1 and not args.quick:
        for mode in (0, 1, 2):
            st.set_hint(mode)
            g_a, g_b = (ga, gb) if mode == hint else (st.graph(st.phase_a), st.graph(st.phase_b))
            by_hint[str(mode)] = {"score_us_per_layer": st.time_graph(g_a, 1, 3) * 1e3 / n_layers,
                                  "select_compact_us_per_layer": st.time_graph(g_b, 1, 3) * 1e3 / n_layers}
        st.set_hint(hint)
        st.phase_a()
        for mode in (0, 1, 2):
            sk.set_select_overlap(mode)
            g_b = gb if mode == sel_overlap else st.graph(st.phase_b)
            by_sel_overlap[str(mode)] = st.time_graph(g_b, 1, 3) * 1e3 / n_layers
        sk.set_select_overlap(sel_overlap)
        st.phase_a(); st.phase_b()                   # leave the caches as the timed step left them
        for mode in (0, 1, 2):
            sk.set_overlap(mode)
            g_c = gc if mode == overlap else st.graph(st.phase_c)
            by_overlap[str(mode)] = st.time_graph(g_c, 8, 3) * 1e3 / (8 * graph_steps * n_layers)
        sk.set_overlap(overlap)
        for variant in (1, 2):                       # 1: mma.sync kernel, 2: tcgen05 kernel (where it applies)
            sk.set_decode_variant(variant)
            by_variant[str(variant)] = st.time_graph(st.graph(st.phase_c), 8, 3) * 1e3 / (8 * graph_steps * n_layers)
        sk.set_decode_variant(args.decode_variant)
    if args.check and rank == 0:
        parity = st.check(O)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ----
    e2e = measure_e2e(args, w, sk, layers, dev, torch)
    e2e["value"] = replicas.max_over_ranks(e2e["value"], dev)
    cpu = cpu_baseline(w, layers[0], torch) if (rank == 0 and args.gpus == 1 and not args.no_cpu_baseline) else None
    st.close()
    del st, layers, ga, gb, gc
    torch.cuda.empty_cache()
    if rank == 0 and args.gpus == 1 and not args.quick:
        for name in ("C4-b1", "C4-b4"):
            other.append(side_workload(B, synth, torch, name, 4, dev, hint, args.check, O))

    peak, peak_kind = measured_peak()
    ab = algorithmic_bytes(w)
    def roof(name, us, kernel, files):
        gbs = ab[name] / (us * 1e-6) / 1e9
        return {"kernel": kernel, "us_per_launch": us, "bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s",
                "frac": gbs / peak, "peak_kind": "of " + peak_kind, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
                "algorithmic_bytes": ab[name], "traffic": ncu_traffic(kernel, files)}
    score_kernel = ("score_logits_kernel+score_finalize_candidates_kernel" if hint == 2
                    else "score_logits_kernel+score_finalize_kernel")
    hf = ["common.cuh", "trace.cuh"]
    kernels = {
        "score": roof("score", a_us, score_kernel, ["score.cu", "select_compact.cu"] + hf),
        "select_compact": roof("select_compact", b_us, "select_compact_kernel", ["select_compact.cu"] + hf),
        "decode_attn": roof("decode_attn", c_us, "decode_attn_kernel", ["decode_attn.cu"] + hf),
    }
    if hint == 2 and w.E >= 14337 and w.k_q > 0:
        # what this mode's select call moves: the candidate lists instead of the score rows (8 tag words and
        # 1.5 k_q + 256 entries of 8 bytes per row at most), the kept rows in and out, the indices
        moved = ab["select_compact"] - w.batch * w.n_q_heads * (w.E * 4 - (32 + 8 * (w.k_q + w.k_q // 2 + 256)))
        kernels["select_compact"]["bytes_moved_in_hint_mode_2"] = moved
        kernels["select_compact"]["frac_of_bytes_moved"] = moved / (b_us * 1e-6) / 1e9 / peak
    if by_hint:
        kernels["select_compact"]["by_hint_mode"] = by_hint
        kernels["select_compact"]["by_select_overlap_mode"] = by_sel_overlap
        kernels["select_compact"]["note"] = ("hint mode 2: sagekv_score leaves a candidate list behind each row and "
                                             "sagekv_select_compact ranks it instead of reading the row, so its DRAM "
                                             "traffic is below the algorithmic bytes (which count the scores); the work "
                                             "moved shows in score_us_per_layer of the same mode")
    if by_overlap:
        kernels["decode_attn"]["by_overlap_mode"] = by_overlap
        kernels["decode_attn"]["by_variant"] = by_variant
    share = {"score": a_us * n_layers, "select_compact": b_us * n_layers, "decode_attn": c_us * c_launches}
    dominant = max(share, key=share.get)

    if rank == 0:
        line = {
            "metric": METRIC, "value": b_us, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": tot_ms, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "shape": "Llama-3.1-8B: %d q / %d kv heads, head_dim %d" % (
                           w.n_q_heads, w.n_kv_heads, w.head_dim),
                       "layers": n_layers, "batch": w.batch, "n_ctx": w.n_ctx, "budget": w.budget, "n_init": w.n_init,
                       "n_recent": w.n_recent, "k_per_kv_head": w.n_sel, "k_q": w.k_q,
                       "decode_steps_per_step": decode_steps, "decode_overlap_mode": overlap, "decode_variant": args.decode_variant, "select_overlap_mode": sel_overlap, "select_hint_mode": hint,
                       "parallelism": "replicas x%d" % args.gpus,
                       "l2": "inputs larger than L2: layers visited round-robin, %.0f MB of K per layer, %.0f MB of "
                             "reduced caches per decode step" % (ab["score"] / 1e6, ab["decode_attn"] * n_layers / 1e6)},
            "score_us_per_layer": a_us, "select_compact_us_per_layer": b_us, "decode_attn_us_per_layer_step": c_us,
            "score_plus_select_compact_us_per_layer": a_us + b_us,
            "decode_attn_hbm_gbs": kernels["decode_attn"]["achieved"],
            "decode_attn_frac_of_peak": kernels["decode_attn"]["frac"],
            "roofline": {k: kernels[dominant][k] for k in ("bound", "achieved", "peak", "unit", "frac", "traffic")},
            "roofline_kernel": kernels[dominant]["kernel"], "roofline_peak_kind": "of " + peak_kind,
            "kernels": kernels,
            "time_share": {k: v / sum(share.values()) for k, v in share.items()},
            "gpu_launches": args.steps * (3 * n_layers + c_launches),
            "wall_ms_per_step": t_wall * 1e3 / args.steps,
            "e2e": e2e, "clocks": clocks,
        }
        for rec in other:
            tag = rec["workload"].lower().replace("-", "_")
            line["select_compact_us_per_layer_" + tag] = rec["select_compact_us_per_layer"]
        if other:
            line["other_workloads"] = other
        if parity is not None:
            line["parity"] = bool(parity and all(r.get("parity", True) for r in other))
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line), flush=True)
    replicas.shutdown()


def measure_e2e(args, w, sk, layers, dev, torch):
    """select+compact per layer with HOST inputs and outputs: pinned scores, K, V in; idx, Kc, Vc out."""
    n_host = min(2, len(layers))
    host = []
    sk.set_select_hint(0)                                # host scores come from anywhere: the plain select path
    for lay in layers[:n_host]:
        host.append({k: lay[k].cpu().pin_memory() for k in ("scores", "K", "V")})
    stage = {"scores": torch.empty_like(layers[0]["scores"]), "K": torch.empty_like(layers[0]["K"]),
             "V": torch.empty_like(layers[0]["V"])}
    cache = sk.new_layer(w.n_init, w.n_recent, w.n_sel)
    out_host = {"idx": torch.empty_like(cache.idx, device="cpu").pin_memory(),
                "Kc": torch.empty_like(cache.Kc, device="cpu").pin_memory(),
                "Vc": torch.empty_like(cache.Vc, device="cpu").pin_memory()}
    h2d = sum(host[0][k].numel() * host[0][k].element_size() for k in host[0])
    d2h = sum(out_host[k].numel() * out_host[k].element_size() for k in out_host)

    def one(i):
        h = host[i % n_host]
        for k in ("scores", "K", "V"):
            stage[k].copy_(h[k], non_blocking=True)
        sk.select_compact(stage["scores"], stage["K"], stage["V"], w.n_init, w.n_recent, w.n_sel, cache)
        out_host["idx"].copy_(cache.idx, non_blocking=True)
        out_host["Kc"].copy_(cache.Kc, non_blocking=True)
        out_host["Vc"].copy_(cache.Vc, non_blocking=True)

    n_per_step = 2
    for i in range(3):
        one(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(args.steps):
        for i in range(n_per_step):
            one(i)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (args.steps * n_per_step)
    full_copy_out = {k: out_host[k].clone() for k in out_host}

    # The same call with K and V left where they are: pinned host memory is addressable from the device, and the
    # kernel reads only the rows it keeps (scores still travel whole).  Reported beside the full-copy figure.
    def one_in_place(i):
        h = host[i % n_host]
        stage["scores"].copy_(h["scores"], non_blocking=True)
        sk.select_compact(stage["scores"], h["K"], h["V"], w.n_init, w.n_recent, w.n_sel, cache)
        out_host["idx"].copy_(cache.idx, non_blocking=True)
        out_host["Kc"].copy_(cache.Kc, non_blocking=True)
        out_host["Vc"].copy_(cache.Vc, non_blocking=True)

    for i in range(3):
        one_in_place(i)
    torch.cuda.synchronize()
    e0.record()
    for s in range(args.steps):
        for i in range(n_per_step):
            one_in_place(i)
    e1.record()
    torch.cuda.synchronize()
    us_in_place = e0.elapsed_time(e1) * 1e3 / (args.steps * n_per_step)
    ok = all(torch.equal(out_host[k], full_copy_out[k]) for k in out_host)   # both ended on the same layer
    rows_bytes = 2 * w.batch * w.n_kv_heads * (w.n_init + w.n_sel + w.n_recent + 1) * w.head_dim * 2
    scores_bytes = host[0]["scores"].numel() * host[0]["scores"].element_size()
    return {"value": us, "unit": UNIT, "h2d_bytes_per_step": h2d * n_per_step, "d2h_bytes_per_step": d2h * n_per_step,
            "layers_per_step": n_per_step,
            "what": "pinned host scores+K+V -> device, sagekv_select_compact, idx+Kc+Vc -> pinned host, per layer",
            "kv_read_in_place": {"value": us_in_place, "unit": UNIT, "outputs_match": bool(ok),
                                 "h2d_bytes_per_step": (scores_bytes + rows_bytes) * n_per_step,
                                 "what": "scores copied, K and V read by the kernel from pinned host memory (kept rows only)"}}


def cpu_baseline(w, lay, torch):
    lay_cpu = {k: lay[k][:1].cpu() for k in ("q_last", "K", "V")}
    t = time_oracle_layer(w, lay_cpu)
    return {"value": t["select_compact_s"] * 1e6, "unit": UNIT, "cores": 1, "kind": "oracle",
            "host_cores": os.cpu_count(),
            "sample": "1 of %d layers of %s: numpy select (lexsort) + row-copy compact, single thread"
                      % (w.n_layers, w.name),
            "score_us_per_layer": t["score_s"] * 1e6, "score_threads": blas_threads(),
            "decode_attn_us_per_layer_step": t["decode_step_s"] * 1e6}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="C3-2048")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (0 = the workload's)")
    ap.add_argument("--decode-steps", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--overlap", type=int, default=None, help="sagekv_set_overlap mode for the decode phase")
    ap.add_argument("--decode-variant", type=int, default=0, help="sagekv_set_decode_variant: 0 library's choice, 1 mma.sync, 2 tcgen05")
    ap.add_argument("--select-overlap", type=int, default=None, help="sagekv_set_select_overlap mode for the select phase")
    ap.add_argument("--hint", type=int, default=2, help="sagekv_set_select_hint mode for the score and select phases")
    ap.add_argument("--check", action="store_true", help="compare layer 0 of every timed workload with the CPU oracle")
    ap.add_argument("--quick", action="store_true", help="only the timed step: no other modes, no other workloads")
    args = ap.parse_args()
    from paper_2503_08879_b200 import synth
    w = synth.workload(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_cuda(args, w)


if __name__ == "__main__":
    main()
