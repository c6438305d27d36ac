"""CUDA path vs the CPU oracle, element by element, through the C-ABI binding.

Tolerances (written out once, used everywhere below):
  scores            |gpu - ref| <= 1e-3 * |ref|            (bf16 products, fp32 sums, approximate exp2)
  selected indices  bit-exact against the oracle's select run on the GPU's own scores; against the
                    oracle's select on the oracle's scores the sets may differ only in tokens whose
                    oracle score is within 1e-3 (relative) of the k-th score
  gathered K, V     bit-exact given the indices
  attention output  |gpu - ref| <= 1e-2 + 1e-2 * |ref|     (bf16 output, bf16 softmax weights)
"""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O
from helpers import bits
from paper_2503_08879_b200 import synth

pytestmark = pytest.mark.gpu

SCORE_RTOL = 1e-3
TIE_BAND = 1e-3
OUT_ATOL, OUT_RTOL = 1e-2, 1e-2


@pytest.fixture(scope="module")
def B():
    from paper_2503_08879_b200 import binding
    return binding


def check_scores(gpu_scores, lay, w, b, scale=None):
    ref = O.score(bits(lay["q_last"][b]), bits(lay["K"][b]), w.n_init, w.n_recent, scale=scale)
    got = gpu_scores.view(w.batch, w.n_q_heads, -1)[b, :, : w.E].cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(got, ref, rtol=SCORE_RTOL, atol=1e-30)
    if w.E > 0:
        np.testing.assert_allclose(got.sum(axis=1), 1.0, atol=1e-4)
    return ref, got


def check_select(idx_gpu, got_scores, ref_scores, w, k_q):
    S = w.n_init
    # (i) same scores in, same indices out
    want = O.select(got_scores.astype(np.float32), k_q, S)
    assert np.array_equal(idx_gpu, want)
    # (ii) against the oracle's own scores: differences only inside the tie band
    ref_idx = O.select(ref_scores.astype(np.float32), k_q, S)
    for h in range(idx_gpu.shape[0]):
        a, r = set(idx_gpu[h].tolist()), set(ref_idx[h].tolist())
        if a == r:
            continue
        kth = np.sort(ref_scores[h])[::-1][k_q - 1]
        for t in a ^ r:
            assert abs(ref_scores[h, t - S] - kth) <= TIE_BAND * kth, (h, t)
    assert np.all(np.diff(idx_gpu, axis=1) > 0)


def check_compact(layer, lay, idx_gpu, w, b):
    Kc_ref, Vc_ref = O.compact(bits(lay["K"][b]), bits(lay["V"][b]), idx_gpu, w.n_init, w.n_recent)
    Kc, Vc = layer.cache()
    assert np.array_equal(bits(Kc[b]), Kc_ref) and np.array_equal(bits(Vc[b]), Vc_ref)
    return Kc_ref, Vc_ref


def check_out(out, ref):
    got = out.float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    assert np.all(err <= OUT_ATOL + OUT_RTOL * np.abs(ref)), float(err.max())


CANARY = 0x5A5A           # bf16 bit pattern in the guard rows of the reduced cache
GUARD_ROWS = 2


def run_pipeline(B, w, n_decode, device="cuda", strided=False, overlap=0, hint=0, scale=0.0, sampled_heads=None, variant=0):
    """All four steps on one layer of workload `w`, every result checked against the oracle.

    Every output buffer carries a guard band (rows behind the reduced cache, floats behind each score row, an
    extra row behind `out`) that must still hold its fill value at the end; score and the first decode step
    run twice and must repeat bit for bit; the context's status word must stay clean.
    sampled_heads: check scores and indices for these query heads only (the oracle's select takes seconds per
    long row); caches and outputs are always checked in full.
    """
    oscale = scale if scale > 0 else None
    lay = synth.make_layer(w, 0, device)
    K, V = lay["K"], lay["V"]
    if strided:   # token stride 136 and a gap between heads: exercises the stride arguments
        Kp = torch.zeros(w.batch, w.n_kv_heads, w.n_ctx + 3, 136, dtype=torch.bfloat16, device=device)
        Vp = torch.zeros_like(Kp)
        Kp[:, :, : w.n_ctx, :128] = K
        Vp[:, :, : w.n_ctx, :128] = V
        K, V = Kp[:, :, : w.n_ctx, :128], Vp[:, :, : w.n_ctx, :128]
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L, softmax_scale=scale)
    sk.set_overlap(overlap)
    sk.set_decode_variant(variant)
    sk.set_select_hint(hint if (hint < 2 or w.n_sel > 0) else 0, w.n_sel)
    stride = sk.score_stride(w.n_ctx, w.n_init, w.n_recent)
    n_rows = w.batch * w.n_q_heads
    buf = torch.full((n_rows, stride + 8), 7.5, dtype=torch.float32, device=device)
    scores = buf[:, :stride]
    B.sagekv_score(sk.ctx, lay["q_last"], K, w.n_ctx, w.n_init, w.n_recent, scores, buf.stride(0))
    first = scores[:, : w.E].clone()
    B.sagekv_score(sk.ctx, lay["q_last"], K, w.n_ctx, w.n_init, w.n_recent, scores, buf.stride(0))
    layer = sk.new_layer(w.n_init, w.n_recent, w.n_sel, spare_rows=GUARD_ROWS)
    layer.Kc.view(torch.int16).fill_(CANARY)
    layer.Vc.view(torch.int16).fill_(CANARY)
    sk.select_compact(scores, K, V, w.n_init, w.n_recent, w.n_sel, layer)
    if hint == 2:                                                     # the same call as a launch whose wait is put off
        sk.set_select_overlap(2)
        ahead = sk.new_layer(w.n_init, w.n_recent, w.n_sel, spare_rows=GUARD_ROWS)
        ahead.Kc.view(torch.int16).fill_(CANARY)
        ahead.Vc.view(torch.int16).fill_(CANARY)
        sk.select_compact(scores, K, V, w.n_init, w.n_recent, w.n_sel, ahead)
        sk.set_select_overlap(0)
        torch.cuda.synchronize()
        assert torch.equal(ahead.idx, layer.idx) and torch.equal(ahead.Kc, layer.Kc) and torch.equal(ahead.Vc, layer.Vc)
    torch.cuda.synchronize()
    assert torch.equal(first, scores[:, : w.E])                       # the score step repeats bit for bit
    if hint == 2 and w.E >= 14337 and 0 < w.k_q <= 2048:                # the lists are there and were usable
        E4 = (w.E + 3) // 4 * 4
        tags = scores[:, E4:E4 + 8].cpu().numpy().view(np.uint32)
        assert (tags[:, 0] == 0x53414732).all() and (tags[:, 1] == w.E).all() and (tags[:, 2] == min(w.k_q, w.E)).all()
        assert (tags[:, 3] >= min(w.k_q, w.E)).mean() >= 0.9, tags[:, 3]   # M = 0 only where the prefilter did not apply
    assert (buf[:, stride:] == 7.5).all()                             # nothing written behind the rows' stride
    if hint == 0:
        assert (buf[:, w.E:] == 7.5).all()
    st = layer.state
    k_q = min(w.k_q, w.E)
    assert (st.n_init, st.k_q, st.n_sel, st.n_recent, st.ring_len, st.len) == (
        w.n_init, k_q, w.G * k_q, w.n_recent, w.n_recent + 1, w.n_init + w.G * k_q + w.n_recent + 1)
    assert int(layer.step.item()) == 0
    heads = list(range(w.n_q_heads)) if sampled_heads is None else list(sampled_heads)
    caches = []
    for b in range(w.batch):
        idx_gpu = layer.indices()[b].cpu().numpy()
        if sampled_heads is None:
            ref_scores, got_scores = check_scores(scores, lay, w, b, oscale)
            if k_q > 0:
                check_select(idx_gpu, got_scores, ref_scores, w, k_q)
        else:
            ref_all = O.score(bits(lay["q_last"][b]), bits(lay["K"][b]), w.n_init, w.n_recent, scale=oscale)
            got_all = scores.view(w.batch, w.n_q_heads, -1)[b, :, : w.E].cpu().numpy().astype(np.float64)
            np.testing.assert_allclose(got_all, ref_all, rtol=SCORE_RTOL, atol=1e-30)
            np.testing.assert_allclose(got_all.sum(axis=1), 1.0, atol=1e-4)
            check_select(idx_gpu[heads], got_all[heads], ref_all[heads], w, k_q)
            assert np.all(np.diff(idx_gpu, axis=1) > 0) and idx_gpu.min() >= w.n_init and idx_gpu.max() < w.n_init + w.E
        caches.append(list(check_compact(layer, lay, idx_gpu, w, b)))
    guard_ok = lambda: bool((layer.Kc[:, :, st.len:].view(torch.int16) == CANARY).all()
                            and (layer.Vc[:, :, st.len:].view(torch.int16) == CANARY).all())
    assert guard_ok()
    # attention with the last token's query and no append, then decode steps with appends
    lse = torch.empty(w.batch, w.n_q_heads, dtype=torch.float32, device=device)
    outbuf = torch.full((w.batch + 1, w.n_q_heads, w.head_dim), 3.0, dtype=torch.bfloat16, device=device)
    out = outbuf[: w.batch]
    sk.decode_attn(lay["q_last"], None, None, layer, out=out, lse=lse)
    torch.cuda.synchronize()
    again = torch.empty_like(out)
    sk.decode_attn(lay["q_last"], None, None, layer, out=again)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), again.view(torch.int16))   # decode repeats bit for bit
    for b in range(w.batch):
        ref, ref_lse, _ = O.decode_step(bits(lay["q_last"][b]), None, None, caches[b][0], caches[b][1], 0,
                                        w.n_init, k_q, w.n_recent, scale=oscale)
        check_out(out[b], ref)
        np.testing.assert_allclose(lse[b].cpu().numpy(), ref_lse, rtol=1e-3, atol=1e-3)
    steps = [0] * w.batch
    for t in range(n_decode):
        d = synth.make_decode_inputs(w, 0, t, device)
        sk.decode_attn(d["q"], d["k_new"], d["v_new"], layer, out=out)
        torch.cuda.synchronize()
        assert int(layer.step.item()) == t + 1
        for b in range(w.batch):
            ref, _, steps[b] = O.decode_step(bits(d["q"][b]), bits(d["k_new"][b]), bits(d["v_new"][b]),
                                             caches[b][0], caches[b][1], steps[b], w.n_init, k_q, w.n_recent,
                                             scale=oscale)
            check_out(out[b], ref)
    Kc, Vc = layer.cache()
    for b in range(w.batch):   # the window rolled the same way on both sides
        assert np.array_equal(bits(Kc[b]), caches[b][0]) and np.array_equal(bits(Vc[b]), caches[b][1])
    assert guard_ok() and bool((outbuf[w.batch] == 3.0).all())
    assert sk.status() == 0
    sk.close()
    return lay, layer


def test_c1_full_config(B):
    w = synth.workload("C1")
    run_pipeline(B, w, n_decode=w.decode_steps)


@pytest.mark.parametrize("name,kw,n_decode", [
    # several score chunks, several cluster CTAs, ragged tails everywhere
    ("C2", dict(n_ctx=20011), 5),
    # window shorter than the number of decode steps: the ring wraps twice
    ("C1", dict(n_ctx=3001, budget=128, n_recent_min=8), 21),
    # G = 7 with the non-divisible budget split, near-duplicate keys (ties at the threshold), batch 2
    ("C4-b1", dict(n_ctx=9000, batch=2), 4),
    # clustered heavy tokens: one CTA of the cluster owns most of the kept rows
    ("C5-4096", dict(n_ctx=30000, budget=1024, n_recent_min=64), 3),
    # reduced cache longer than one partition pass: several tiles per CTA in decode
    ("C3-4096", dict(n_ctx=40000), 3),
    # k_q too large for the prefilter (radix path at scale) and a reduced cache long enough for several
    # clusters per KV head in decode (partition results merged through scratch)
    ("C3-4096", dict(n_ctx=30000, budget=12600), 2),
    # clustered heavy tokens with a large budget: hundreds of kept rows in one CTA of the select cluster
    ("C5-8192", dict(n_ctx=60000, budget=4096, n_recent_min=64), 2),
    # more (batch, KV head) pairs than clusters of 8 fit at once: decode runs with clusters of 6 (20 pairs) and
    # of 5 (24 pairs), whose CTAs finish unequal shares of the 128 output columns
    ("C4-b1", dict(n_ctx=6000, batch=5), 2),
    ("C4-b1", dict(n_ctx=6000, batch=6), 2),
    # many score rows (112) that carry the score step's group maxima: select runs with clusters of 2, unstaged
    ("C4-b1", dict(n_ctx=20000, batch=4), 1),
    # and 56 rows: clusters of 4
    ("C4-b1", dict(n_ctx=20000, batch=2), 1),
])
@pytest.mark.parametrize("hint", [0, 1, 2])
def test_scaled_configs(B, name, kw, n_decode, hint):
    w = synth.workload(name).with_(n_layers=1, **kw)
    run_pipeline(B, w, n_decode, hint=hint)


@pytest.mark.parametrize("name,kw,n_decode,overlap", [
    ("C1", dict(), 8, 0),                                                   # 33 tiles: five per CTA, one score block
    ("C1", dict(n_ctx=3001, budget=128, n_recent_min=8), 21, 1),            # the ring wraps twice
    ("C3-2048", dict(n_ctx=20011), 4, 0),                                    # 129 tiles: the benchmark's geometry, three blocks
    ("C2", dict(n_ctx=20011), 5, 2),
    ("C4-b1", dict(n_ctx=9000, batch=2), 4, 0),                              # G = 7
    ("C4-b1", dict(n_ctx=6000, batch=5), 2, 0),                              # clusters of 6: unequal column shares
    ("C1", dict(n_ctx=300, budget=24, n_init=4, n_recent_min=20), 3, 0),     # k = 0: sink + recent only
    ("C1", dict(n_ctx=2, budget=1, n_init=0, n_recent_min=1), 3, 0),         # two tokens: a single tile
    ("C3-4096", dict(n_ctx=40000), 3, 0),                                    # beyond the variant's reach: runs as variant 1
])
def test_decode_tensor_memory_variant(B, name, kw, n_decode, overlap):
    """sagekv_set_decode_variant(2): both products on tcgen05 with accumulators in tensor memory; same oracle,
    same tolerance."""
    w = synth.workload(name).with_(n_layers=1, **kw)
    run_pipeline(B, w, n_decode, overlap=overlap, variant=2)


def test_strided_cache(B):
    w = synth.workload("C1").with_(n_ctx=5000)
    run_pipeline(B, w, 3, strided=True)


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 4), (16, 2), (8, 1)])
def test_group_sizes(B, hq, hkv):
    w = synth.workload("C1").with_(n_q_heads=hq, n_kv_heads=hkv, n_ctx=2500, budget=4 + 8 * (hq // hkv) + 16,
                                   n_recent_min=16)
    run_pipeline(B, w, 3)


@pytest.mark.parametrize("kw", [
    dict(n_ctx=70, budget=72, n_init=4, n_recent_min=64),      # E = 1, k_q = 1
    dict(n_ctx=69, budget=72, n_init=4, n_recent_min=64),      # E = 0: the cache is everything
    dict(n_ctx=100, budget=228, n_init=4, n_recent_min=64),    # k_q = 40 > E = 31: clamped, k_q = E
    dict(n_ctx=300, budget=24, n_init=4, n_recent_min=20),     # k = 0: sink + recent only
    dict(n_ctx=300, budget=36, n_init=0, n_recent_min=0),      # no sink, no recent window (ring of 1)
    dict(n_ctx=2, budget=1, n_init=0, n_recent_min=1),         # two tokens
])
def test_degenerate_partitions(B, kw):
    w = synth.workload("C1").with_(**kw)
    run_pipeline(B, w, 3)


def test_full_size_128k_one_layer(B):
    """C3 at budget 2048, one layer, the launch configuration the benchmark times."""
    w = synth.workload("C3-2048")
    run_pipeline(B, w, 2, hint=1)


@pytest.mark.parametrize("name,hint", [
    ("C2", 0),          # 32K context
    ("C3-1024", 1),     # 128K, the smaller and the larger budget
    ("C3-2048", 0),
    ("C3-4096", 0),
    ("C4-b1", 1),       # Qwen shape, G = 7
    ("C5-4096", 0),     # 512K: the select step reads its unstaged slice in four rounds, the score grid has 2047 chunks
    ("C5-4096", 1),
    ("C5-8192", 1),
    ("C3-2048", 2),     # and starting from the candidate lists the score step leaves behind the rows
    ("C4-b1", 2),
    ("C5-4096", 2),
    ("C5-8192", 2),
])
def test_every_workload_at_full_size_one_layer(B, name, hint):
    """Each workload at its full context and budget, one layer, with and without the hint behind the score
    rows: scores, indices, reduced cache, two decode steps, all against the oracle."""
    w = synth.workload(name).with_(n_layers=1)
    run_pipeline(B, w, 2, hint=hint)


@pytest.mark.parametrize("sel_overlap", [0, 2])
def test_candidate_lists_with_a_large_group_of_equal_scores_at_the_cut(B, sel_overlap):
    """Hint mode 2 on rows in which several hundred tokens share one key, placed so that the k-th score falls
    inside that group: the select step starts from the score step's list, finds too many equal scores at the cut
    for its exact ranking and hands the row to the radix path.  The lowest positions of the group must be kept."""
    w = synth.workload("C2").with_(n_ctx=30001, n_layers=1, budget=4 + 128 + 4 * 300, structure="count", heavy=(100,))
    dev = "cuda"
    lay = synth.make_layer(w, 0, dev)
    g = torch.Generator(device=dev).manual_seed(77)
    for kvh in range(w.n_kv_heads):                      # 800 copies of one strong key per KV head
        pos = torch.randperm(w.E, generator=g, device=dev)[:800] + w.n_init
        q_hat = lay["q_last"][0, kvh * w.G].float()
        q_hat = q_hat / q_hat.norm()
        lay["K"][0, kvh, pos] = (3.0 * q_hat).to(torch.bfloat16)
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, 1, max_ctx=w.n_ctx, max_len=w.L)
    sk.set_select_overlap(sel_overlap)                    # 2: the launch whose wait is put off, falling back after it
    for hint, spoil in ((2, False), (2, True), (0, False)):
        sk.set_select_hint(hint, w.n_sel)
        scores = sk.score(lay["q_last"], lay["K"], w.n_init, w.n_recent)
        if spoil:                                        # rows without a usable list: the tag's first word says so
            E4 = (w.E + 3) // 4 * 4
            scores[::3, E4:E4 + 1] = 0.0
        layer = sk.select_compact(scores, lay["K"], lay["V"], w.n_init, w.n_recent, w.n_sel)
        layer2 = sk.select_compact(scores, lay["K"], lay["V"], w.n_init, w.n_recent, w.n_sel)   # back to back
        torch.cuda.synchronize()
        got = scores[:, : w.E].cpu().numpy()
        for lyr in (layer, layer2):
            idx = lyr.indices()[0].cpu().numpy()
            assert np.array_equal(idx, O.select(got, w.k_q, w.n_init)), (hint, spoil)
            check_compact(lyr, lay, idx, w, 0)
    assert sk.status() == 0
    sk.close()


@pytest.mark.parametrize("scale", [0.05, 0.2])
def test_softmax_scale_override(B, scale):
    """A context created with its own softmax scale instead of 1/sqrt(d): score and decode must both use it."""
    w = synth.workload("C2").with_(n_ctx=9001, n_layers=1, budget=516)
    run_pipeline(B, w, 3, scale=scale)
    w = synth.workload("C4-b1").with_(n_ctx=16500, n_layers=1, batch=2)
    run_pipeline(B, w, 2, scale=scale, hint=1)


def test_full_size_qwen_128k_batch4_sampled(B):
    """C4 at batch 4: scores and indices checked for one batch entry, caches and outputs for all."""
    w = synth.workload("C4-b4")
    dev = "cuda"
    lay = synth.make_layer(w, 0, dev)
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L)
    sk.set_select_hint(1)
    scores = sk.score(lay["q_last"], lay["K"], w.n_init, w.n_recent)
    layer = sk.select_compact(scores, lay["K"], lay["V"], w.n_init, w.n_recent, w.n_sel)
    d = synth.make_decode_inputs(w, 0, 0, dev)
    out = sk.decode_attn(d["q"], d["k_new"], d["v_new"], layer)
    torch.cuda.synchronize()
    for b in range(w.batch):
        idx_gpu = layer.indices()[b].cpu().numpy()
        got = scores.view(w.batch, w.n_q_heads, -1)[b, :, : w.E].cpu().numpy()
        assert np.array_equal(idx_gpu, O.select(got, w.k_q, w.n_init))
        if b == 3:
            ref_scores, got_scores = check_scores(scores, lay, w, b)
            check_select(idx_gpu, got_scores, ref_scores, w, w.k_q)
        Kc_ref, Vc_ref = O.compact(bits(lay["K"][b]), bits(lay["V"][b]), idx_gpu, w.n_init, w.n_recent)
        ref, _, _ = O.decode_step(bits(d["q"][b]), bits(d["k_new"][b]), bits(d["v_new"][b]), Kc_ref, Vc_ref, 0,
                                  w.n_init, w.k_q, w.n_recent)
        check_out(out[b], ref)
        Kc, Vc = layer.cache()
        assert np.array_equal(bits(Kc[b]), Kc_ref) and np.array_equal(bits(Vc[b]), Vc_ref)
    sk.close()


def test_dependent_launch_same_layer_back_to_back(B):
    """Overlap mode 1 (wait before touching anything) must be right for any predecessor, here the previous
    step of the same layer, issued without host synchronisation in between."""
    w = synth.workload("C1").with_(n_ctx=3001, budget=128, n_recent_min=8)
    run_pipeline(B, w, 12, overlap=1)
    dev = "cuda"
    lay = synth.make_layer(w, 0, dev)
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L)
    sk.set_overlap(1)
    scores = sk.score(lay["q_last"], lay["K"], w.n_init, w.n_recent)
    layer = sk.select_compact(scores, lay["K"], lay["V"], w.n_init, w.n_recent, w.n_sel)
    torch.cuda.synchronize()
    idx = layer.indices()[0].cpu().numpy()
    Kc_ref, Vc_ref = O.compact(bits(lay["K"][0]), bits(lay["V"][0]), idx, w.n_init, w.n_recent)
    n = 25
    ins = [synth.make_decode_inputs(w, 0, t, dev) for t in range(n)]
    outs = [torch.empty_like(ins[0]["q"]) for _ in range(n)]
    for t in range(n):                                   # no synchronisation between the launches
        sk.decode_attn(ins[t]["q"], ins[t]["k_new"], ins[t]["v_new"], layer, outs[t])
    torch.cuda.synchronize()
    step = 0
    for t in range(n):
        ref, _, step = O.decode_step(bits(ins[t]["q"][0]), bits(ins[t]["k_new"][0]), bits(ins[t]["v_new"][0]),
                                     Kc_ref, Vc_ref, step, w.n_init, w.k_q, w.n_recent)
        check_out(outs[t][0], ref)
    assert int(layer.step.item()) == n
    sk.close()


@pytest.mark.parametrize("mode,hint", [(1, 0), (1, 2), (2, 2), (2, 1), (2, 0)])
def test_select_overlap_across_layers(B, mode, hint):
    """sagekv_set_select_overlap: the select calls of three layers follow one another on the stream, several rounds
    without host synchronisation, after the score calls of all layers (so no call's predecessor writes its inputs,
    which is what mode 2 asks for; with hint 2 the selection then runs ahead of the dependency wait).  Indices are
    those of the oracle's select on the GPU's scores, caches are the oracle's gather, the step words are reset."""
    w = synth.workload("C3-2048").with_(n_ctx=20011, n_layers=3)
    dev = "cuda"
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L)
    sk.set_select_hint(hint, w.n_sel)
    stride = sk.score_stride(w.n_ctx, w.n_init, w.n_recent)
    lays, caches, scores = [], [], []
    for l in range(3):
        lay = synth.make_layer(w, l, dev)
        sc = sk.new_scores(w.n_ctx, w.n_init, w.n_recent)
        B.sagekv_score(sk.ctx, lay["q_last"], lay["K"], w.n_ctx, w.n_init, w.n_recent, sc, stride)
        c = sk.new_layer(w.n_init, w.n_recent, w.n_sel, spare_rows=GUARD_ROWS)
        lays.append(lay); scores.append(sc); caches.append(c)
    sk.set_select_overlap(mode)
    for rnd in range(3):
        for c in caches:
            c.Kc.view(torch.int16).fill_(CANARY)
            c.Vc.view(torch.int16).fill_(CANARY)
            c.idx.fill_(-1)
            c.step.fill_(99)
        for l in range(3):                                # back to back: nothing between the three launches
            sk.select_compact(scores[l], lays[l]["K"], lays[l]["V"], w.n_init, w.n_recent, w.n_sel, caches[l])
    torch.cuda.synchronize()
    assert sk.status() == 0
    for l in range(3):
        got = scores[l].view(w.batch, w.n_q_heads, -1)[0, :, : w.E].cpu().numpy()
        idx = caches[l].indices()[0].cpu().numpy()
        assert np.array_equal(idx, O.select(got, w.k_q, w.n_init))
        Kc_ref, Vc_ref = O.compact(bits(lays[l]["K"][0]), bits(lays[l]["V"][0]), idx, w.n_init, w.n_recent)
        Kc, Vc = caches[l].cache()
        assert np.array_equal(bits(Kc[0]), Kc_ref) and np.array_equal(bits(Vc[0]), Vc_ref)
        assert (caches[l].Kc.view(torch.int16)[:, :, w.L:] == CANARY).all()
        assert int(caches[l].step.item()) == 0
    sk.close()


def test_prefetch_overlap_across_layers(B):
    """Overlap mode 2: decode calls of different layers alternate on one stream, so the kernel before each
    call never writes that call's cache, which is what the mode asks the caller to guarantee."""
    w = synth.workload("C2").with_(n_ctx=6000, n_layers=3)
    dev = "cuda"
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L)
    layers, refs = [], []
    for l in range(3):
        lay = synth.make_layer(w, l, dev)
        scores = sk.score(lay["q_last"], lay["K"], w.n_init, w.n_recent)
        layer = sk.select_compact(scores, lay["K"], lay["V"], w.n_init, w.n_recent, w.n_sel)
        torch.cuda.synchronize()
        idx = layer.indices()[0].cpu().numpy()
        refs.append(list(O.compact(bits(lay["K"][0]), bits(lay["V"][0]), idx, w.n_init, w.n_recent)))
        layers.append(layer)
    sk.set_overlap(2)
    n = 6
    ins = [[synth.make_decode_inputs(w, l, t, dev) for l in range(3)] for t in range(n)]
    outs = [[torch.empty_like(ins[0][0]["q"]) for _ in range(3)] for _ in range(n)]
    for t in range(n):
        for l in range(3):
            d = ins[t][l]
            sk.decode_attn(d["q"], d["k_new"], d["v_new"], layers[l], outs[t][l])
    torch.cuda.synchronize()
    steps = [0, 0, 0]
    for t in range(n):
        for l in range(3):
            d = ins[t][l]
            ref, _, steps[l] = O.decode_step(bits(d["q"][0]), bits(d["k_new"][0]), bits(d["v_new"][0]),
                                             refs[l][0], refs[l][1], steps[l], w.n_init, w.k_q, w.n_recent)
            check_out(outs[t][l][0], ref)
    for l in range(3):
        Kc, Vc = layers[l].cache()
        assert np.array_equal(bits(Kc[0]), refs[l][0]) and np.array_equal(bits(Vc[0]), refs[l][1])
    sk.close()
