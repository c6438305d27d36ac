"""The synthetic generator: shapes, determinism and the planted structure."""

import numpy as np
import torch

from paper_2503_08879_b200 import synth


def small(name, **kw):
    base = dict(n_layers=1, n_ctx=600, decode_steps=2)
    base.update(kw)
    return synth.workload(name).with_(**base)


def test_workload_table_matches_budget_arithmetic():
    w = synth.workload("C1")
    assert (w.n_init, w.n_recent, w.n_sel, w.k_q, w.E, w.L) == (4, 64, 444, 111, 4027, 513)
    w = synth.workload("C3-2048")
    assert (w.n_recent, w.n_sel, w.k_q, w.E, w.L) == (128, 1916, 479, 130939, 2049)
    w = synth.workload("C4-b1")           # G = 7: remainder slots go to the recent window
    assert (w.G, w.k_q, w.n_sel, w.n_recent, w.E, w.L) == (7, 273, 1911, 133, 130934, 2049)
    w = synth.workload("C5-8192")
    assert (w.n_recent, w.k_q, w.n_sel, w.L) == (256, 1983, 7932, 8193)
    for w in synth.WORKLOADS.values():
        assert w.n_init + w.n_sel + w.n_recent == w.budget
        assert w.n_init + w.E + w.n_recent + 1 == w.n_ctx


def test_make_layer_is_deterministic_and_shaped():
    w = small("C1", budget=64, n_recent_min=8)
    a, b = synth.make_layer(w, 0), synth.make_layer(w, 0)
    assert a["K"].shape == (1, 8, 600, 128) and a["K"].dtype == torch.bfloat16
    assert a["q_last"].shape == (1, 32, 128)
    for key in ("q_last", "K", "V"):
        assert torch.equal(a[key].view(torch.int16), b[key].view(torch.int16))
    c = synth.make_layer(w, 1)
    assert not torch.equal(a["K"].view(torch.int16), c["K"].view(torch.int16))


def test_heavy_tokens_sit_in_eviction_region_and_align_with_their_query():
    w = small("C1", budget=64, n_recent_min=8)
    lay = synth.make_layer(w, 0)
    q = lay["q_last"][0].float()
    for g in range(w.n_kv_heads):
        pos = lay["heavy"][0][g]
        assert pos.numel() == 32 and pos.min() >= w.n_init and pos.max() < w.n_init + w.E
        for j, t in enumerate(pos.tolist()):
            h = g * w.G + j % w.G
            cos = torch.nn.functional.cosine_similarity(lay["K"][0, g, t].float(), q[h], dim=0)
            assert cos > 0.4


def test_dups_structure_creates_exact_ties():
    w = small("C4-b1", n_ctx=3000, budget=256, n_recent_min=16)
    lay = synth.make_layer(w, 0)
    K = lay["K"][0, 0].view(torch.int16).numpy()
    rows = {}
    dup = 0
    for t in range(w.n_init, w.n_init + w.E):
        key = K[t].tobytes()
        dup += key in rows
        rows[key] = t
    assert dup >= 2


def test_spans_structure_is_contiguous():
    w = small("C5-4096", n_ctx=5000, budget=256, n_recent_min=16)
    pos = np.sort(synth.make_layer(w, 0)["heavy"][0][0].numpy())
    runs = 1 + int((np.diff(pos) > 1).sum())
    assert runs <= 8 and pos.size >= 8


def test_decode_inputs():
    w = small("C1")
    a, b = synth.make_decode_inputs(w, 0, 3), synth.make_decode_inputs(w, 0, 3)
    assert a["q"].shape == (1, 32, 128) and a["k_new"].shape == (1, 8, 128)
    assert torch.equal(a["v_new"].view(torch.int16), b["v_new"].view(torch.int16))
