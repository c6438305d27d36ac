"""The comparison paths beside the four steps, against the oracle: StreamLLM_R's cache (pre-RoPE keys rotated by
their index inside the kept window while they are gathered; Section 3.1 "Baselines", Appendix A.1), StreamLLM with
absolute positions (the k = 0 case of the ordinary calls), and the pooled reading of Step 2 (one selection per KV
head from the summed score rows of its query heads).

Tolerances: rotated keys are computed in double precision on both sides and rounded once to bf16; the two roundings
(fp64 -> bf16 in the oracle, fp64 -> fp32 -> bf16 on the GPU) can differ by one bf16 unit in the last place at
rounding ties, so rows must agree bit for bit on at least 99.9 % of the elements and within one unit elsewhere.
Pooled scores: relative 1e-3 (fp32 sums of four to eight fp32 terms); indices bit-exact on the GPU's own pooled
scores; attention output 1e-2 + 1e-2 relative as everywhere."""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O
from helpers import bits
from paper_2503_08879_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2503_08879_b200 import binding
    return binding


def check_out(out, ref):
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= 1e-2 + 1e-2 * np.abs(ref)), float(np.abs(got - ref).max())


@pytest.mark.parametrize("N,S,R,theta,batch", [(5000, 4, 128, 10000.0, 1), (131072, 4, 2043, 500000.0, 1),
                                                (300, 0, 17, 10000.0, 2), (70, 64, 5, 1000000.0, 1)])
def test_streamllm_r_cache_matches_the_oracle(B, N, S, R, theta, batch):
    Hq, Hkv = 8, 2
    g = torch.Generator(device="cuda").manual_seed(N + R)
    K = torch.randn(batch, Hkv, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    V = torch.randn(batch, Hkv, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    L = S + R + 1
    sk = B.SageKV(Hq, Hkv, 128, batch, max_ctx=N, max_len=L)
    layer = sk.new_layer(S, R, 0, spare_rows=2)
    layer.Kc.view(torch.int16).fill_(0x5A5A)
    layer.Vc.view(torch.int16).fill_(0x5A5A)
    B.sagekv_compact_window_rope(sk.ctx, K, V, N, S, R, theta, layer.Kc, layer.Vc, layer.state)
    torch.cuda.synchronize()
    st = layer.state
    assert (st.n_init, st.k_q, st.n_sel, st.n_recent, st.ring_len, st.len) == (S, 0, 0, R, R + 1, L)
    assert int(layer.step.item()) == 0
    assert (layer.Kc[:, :, L:].view(torch.int16) == 0x5A5A).all() and (layer.Vc[:, :, L:].view(torch.int16) == 0x5A5A).all()
    caches = []
    for b in range(batch):
        Kc_ref, Vc_ref = O.compact_window_rope(bits(K[b]), bits(V[b]), S, R, theta)
        got_k, got_v = bits(layer.Kc[b, :, :L]), bits(layer.Vc[b, :, :L])
        assert np.array_equal(got_v, Vc_ref)
        same = got_k == Kc_ref
        assert same.mean() >= 0.999
        ulp_off = np.abs(got_k.astype(np.int32) - Kc_ref.astype(np.int32))
        assert ulp_off.max() <= 1
        if S > 0:
            assert np.array_equal(got_k[:, 0], bits(K[b, :, 0]))        # position 0 is not rotated
        caches.append((got_k.copy(), got_v.copy()))
    # decode on the rotated cache runs as on any reduced cache (no selected segment)
    q = torch.randn(batch, Hq, 128, generator=g, device="cuda").to(torch.bfloat16)
    out = sk.decode_attn(q, None, None, layer)
    torch.cuda.synchronize()
    for b in range(batch):
        ref, _, _ = O.decode_step(bits(q[b]), None, None, caches[b][0], caches[b][1], 0, S, 0, R)
        check_out(out[b], ref)
    assert sk.status() == 0
    sk.close()


def test_streamllm_abs_is_the_k0_case(B):
    """StreamLLM with absolute positions keeps sink + recent of the ordinary (already rotated) cache: k = 0."""
    w = synth.workload("C2").with_(n_ctx=9000, n_layers=1, budget=4 + 200, n_recent_min=200)
    assert w.n_sel == 0
    lay = synth.make_layer(w, 0, "cuda")
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, 128, 1, max_ctx=w.n_ctx, max_len=w.L)
    layer = sk.select_compact(None, lay["K"], lay["V"], w.n_init, w.n_recent, 0)
    d = synth.make_decode_inputs(w, 0, 0, "cuda")
    out = sk.decode_attn(d["q"], d["k_new"], d["v_new"], layer)
    torch.cuda.synchronize()
    Kb, Vb = bits(lay["K"][0]), bits(lay["V"][0])
    rows = list(range(w.n_init)) + list(range(w.n_ctx - 1 - w.n_recent, w.n_ctx))
    Kc_ref, Vc_ref = Kb[:, rows].copy(), Vb[:, rows].copy()
    ref, _, _ = O.decode_step(bits(d["q"][0]), bits(d["k_new"][0]), bits(d["v_new"][0]), Kc_ref, Vc_ref, 0, w.n_init, 0,
                              w.n_recent)
    check_out(out[0], ref)
    sk.close()


@pytest.mark.parametrize("name,kw,K_sel", [("C2", dict(n_ctx=20011), 1916), ("C4-b1", dict(n_ctx=30000, batch=2), 1900),
                                            ("C1", dict(n_ctx=3001), 37)])
def test_pooled_group_mode_matches_the_oracle(B, name, kw, K_sel):
    w = synth.workload(name).with_(n_layers=1, **kw)
    dev = "cuda"
    lay = synth.make_layer(w, 0, dev)
    S, R, G = w.n_init, w.n_recent, w.G
    L = S + K_sel + R + 1
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, 128, w.batch, max_ctx=w.n_ctx, max_len=L)
    scores = sk.score(lay["q_last"], lay["K"], S, R)
    E4 = (w.E + 3) // 4 * 4
    pooled = torch.full((w.batch * w.n_kv_heads, E4 + 4), 7.5, dtype=torch.float32, device=dev)
    B.sagekv_pool_scores(sk.ctx, scores, scores.stride(0), w.n_ctx, S, R, pooled, pooled.stride(0))
    B.sagekv_set_group_mode(sk.ctx, 1)
    layer = B.Layer(w.batch, w.n_kv_heads, w.n_kv_heads, 128, L, K_sel, torch.device(dev))   # idx: one list per KV head
    B.sagekv_select_compact(sk.ctx, pooled, pooled.stride(0), lay["K"], lay["V"], w.n_ctx, S, R, K_sel, layer.idx,
                            layer.Kc, layer.Vc, layer.state)
    d = synth.make_decode_inputs(w, 0, 0, dev)
    out = torch.empty_like(d["q"])
    B.sagekv_decode_attn(sk.ctx, d["q"], d["k_new"], d["v_new"], layer.Kc, layer.Vc, layer.state, out)
    torch.cuda.synchronize()
    assert (pooled[:, w.E:] == 7.5).all()
    st = layer.state
    assert (st.k_q, st.n_sel, st.len) == (K_sel, K_sel, L)
    for b in range(w.batch):
        p = scores.view(w.batch, w.n_q_heads, -1)[b, :, : w.E].cpu().numpy()
        got_pool = pooled.view(w.batch, w.n_kv_heads, -1)[b, :, : w.E].cpu().numpy()
        want_pool = p.reshape(w.n_kv_heads, G, w.E).astype(np.float64).sum(axis=1)
        np.testing.assert_allclose(got_pool, want_pool, rtol=1e-3, atol=1e-30)
        idx = layer.idx.flatten()[: w.batch * w.n_kv_heads * K_sel].view(w.batch, w.n_kv_heads, K_sel)[b].cpu().numpy()
        assert np.array_equal(idx, O.select(got_pool, K_sel, S))             # bit-exact on the GPU's own pooled scores
        ref_idx = O.select_pooled(p, K_sel, S, G)                            # against the oracle's pooling: ties only
        for g in range(w.n_kv_heads):
            diff = set(idx[g].tolist()) ^ set(ref_idx[g].tolist())
            kth = np.sort(want_pool[g])[::-1][K_sel - 1]
            assert all(abs(want_pool[g, t - S] - kth) <= 1e-3 * kth for t in diff)
        Kc_ref, Vc_ref = O.compact_pooled(bits(lay["K"][b]), bits(lay["V"][b]), idx, S, R)
        ref, _, _ = O.decode_step_pooled(bits(d["q"][b]), bits(d["k_new"][b]), bits(d["v_new"][b]), Kc_ref, Vc_ref, 0, S,
                                         K_sel, R)                             # (appends the new token to Kc_ref, Vc_ref)
        assert np.array_equal(bits(layer.Kc[b, :, :L]), Kc_ref) and np.array_equal(bits(layer.Vc[b, :, :L]), Vc_ref)
        check_out(out[b], ref)
    assert sk.status() == 0
    sk.close()


@pytest.mark.parametrize("name,kw", [("C1", dict()), ("C4-b1", dict(n_ctx=20000, batch=2)), ("C2", dict(n_ctx=32768 - 7))])
def test_quest_style_block_selection_matches_the_oracle(B, name, kw):
    """Block summaries bit-exact (minima and maxima of bf16 values are not rounded), bounds within 1e-3 of the sum of
    the absolute terms (fp32 sums of 128 products), block selection bit-exact on the GPU's own bounds and, against
    the oracle's bounds, different only for blocks whose bound is within that tolerance of the cut."""
    w = synth.workload(name).with_(n_layers=1, **kw)
    dev = "cuda"
    lay = synth.make_layer(w, 0, dev)
    S, R, E = w.n_init, w.n_recent, w.E
    nb = (E + 15) // 16
    keep = max(1, w.k_q // 16)
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, 128, w.batch, max_ctx=w.n_ctx, max_len=w.L)
    kmin = torch.full((w.batch, w.n_kv_heads, nb + 1, 128), 3.0, dtype=torch.bfloat16, device=dev)
    kmax = torch.full_like(kmin, 3.0)
    B.sagekv_quest_build(sk.ctx, lay["K"], w.n_ctx, S, R, kmin, kmax)
    torch.cuda.synchronize()
    # the kernel writes [batch, H_kv, nb, 128] contiguous: view the buffers that way
    km = kmin.flatten()[: w.batch * w.n_kv_heads * nb * 128].view(w.batch, w.n_kv_heads, nb, 128)
    kM = kmax.flatten()[: w.batch * w.n_kv_heads * nb * 128].view(w.batch, w.n_kv_heads, nb, 128)
    assert (kmin.flatten()[w.batch * w.n_kv_heads * nb * 128:] == 3.0).all()             # nothing written behind
    stride = (nb + 3) // 4 * 4
    u = torch.full((w.batch * w.n_q_heads, stride), 7.5, dtype=torch.float32, device=dev)
    B.sagekv_quest_bounds(sk.ctx, lay["q_last"], km, kM, nb, u, stride)
    idx = torch.full((w.batch * w.n_q_heads, keep + 1), -7, dtype=torch.int32, device=dev)
    B.sagekv_select_topk(sk.ctx, u, stride, nb, keep, idx.flatten()[: w.batch * w.n_q_heads * keep].view(-1, keep))
    torch.cuda.synchronize()
    assert (u[:, nb:] == 7.5).all()
    got_idx = idx.flatten()[: w.batch * w.n_q_heads * keep].view(w.batch, w.n_q_heads, keep).cpu().numpy()
    assert (idx.flatten()[w.batch * w.n_q_heads * keep:] == -7).all()
    for b in range(w.batch):
        rmin, rmax = O.quest_summaries(bits(lay["K"][b]), S, R)
        assert np.array_equal(bits(km[b]), rmin) and np.array_equal(bits(kM[b]), rmax)
        ref_u = O.quest_bounds(bits(lay["q_last"][b]), rmin, rmax)
        got_u = u.view(w.batch, w.n_q_heads, stride)[b, :, :nb].cpu().numpy()
        qf = O.bf16_bits_to_f64(bits(lay["q_last"][b]))
        G = w.G
        for h in range(w.n_q_heads):
            mag = np.sum(np.maximum(np.abs(qf[h] * O.bf16_bits_to_f64(rmin[h // G])), np.abs(qf[h] * O.bf16_bits_to_f64(rmax[h // G]))),
                         axis=-1) / np.sqrt(128.0)
            assert np.all(np.abs(got_u[h] - ref_u[h]) <= 1e-3 * mag + 1e-6)
        assert np.array_equal(got_idx[b], O.quest_select(got_u, keep))
        ref_idx = O.quest_select(ref_u, keep)
        for h in range(w.n_q_heads):
            diff = set(got_idx[b, h].tolist()) ^ set(ref_idx[h].tolist())
            cut = np.sort(ref_u[h])[::-1][keep - 1]
            assert all(abs(ref_u[h, j] - cut) <= 2e-3 * max(1.0, abs(cut)) for j in diff)
    assert sk.status() == 0
    sk.close()
