"""Interval-based refresh (the paper's Conclusion: "periodically refreshes selected key tokens").

Nothing new is needed in the library for it: the caller keeps the full cache, appends every generated
token's (k, v) to it, and every so often runs score + select_compact again with the current token's
query on the longer sequence.  This test does exactly that through the C-ABI binding and checks the
refreshed reduced cache and the decode steps after it against the oracle run on the extended sequence.
The recent window needs no special care: the last R+1 tokens of the extended sequence are the rows
the rolling window holds at that moment."""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O
from paper_2503_08879_b200 import synth

pytestmark = pytest.mark.gpu


def bits(t):
    return t.detach().cpu().contiguous().view(torch.uint16).numpy()


def test_refresh_after_decode_equals_pipeline_on_extended_sequence():
    from paper_2503_08879_b200 import binding as B
    dev = "cuda"
    w = synth.workload("C2").with_(n_ctx=6000, n_layers=1, budget=260, n_recent_min=32)
    S, R, k_q, G = w.n_init, w.n_recent, w.k_q, w.G
    T = 2 * (R + 1) + 7                                   # the window wraps twice before the refresh
    N, N2 = w.n_ctx, w.n_ctx + T
    lay = synth.make_layer(w, 0, dev)
    Kf = torch.zeros(1, w.n_kv_heads, N2 + 8, 128, dtype=torch.bfloat16, device=dev)
    Vf = torch.zeros_like(Kf)
    Kf[:, :, :N], Vf[:, :, :N] = lay["K"], lay["V"]
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, 128, 1, max_ctx=N2, max_len=w.L)
    layer = sk.select_compact(sk.score(lay["q_last"], Kf[:, :, :N], S, R), Kf[:, :, :N], Vf[:, :, :N], S, R, w.n_sel)
    for t in range(T):                                    # decode; the caller also grows the full cache
        d = synth.make_decode_inputs(w, 0, t, dev)
        sk.decode_attn(d["q"], d["k_new"], d["v_new"], layer)
        Kf[:, :, N + t], Vf[:, :, N + t] = d["k_new"], d["v_new"]
    torch.cuda.synchronize()
    Kc_old, Vc_old = (x.clone() for x in layer.cache())

    # refresh with the query of the token generated last
    q_cur = d["q"]
    K2, V2 = Kf[:, :, :N2], Vf[:, :, :N2]
    scores2 = sk.score(q_cur, K2, S, R)
    layer2 = sk.select_compact(scores2, K2, V2, S, R, w.n_sel)
    torch.cuda.synchronize()
    E2 = N2 - 1 - S - R
    ref_p = O.score(bits(q_cur[0]), bits(K2[0]), S, R)
    got_p = scores2[:, :E2].cpu().numpy()
    np.testing.assert_allclose(got_p, ref_p, rtol=1e-3, atol=1e-30)
    idx = layer2.indices()[0].cpu().numpy()
    assert np.array_equal(idx, O.select(got_p, k_q, S))
    Kc_ref, Vc_ref = O.compact(bits(K2[0]), bits(V2[0]), idx, S, R)
    Kc2, Vc2 = layer2.cache()
    assert np.array_equal(bits(Kc2[0]), Kc_ref) and np.array_equal(bits(Vc2[0]), Vc_ref)
    assert int(layer2.step.item()) == 0
    # the window of the refreshed cache holds the same rows as the rolled window before the refresh
    win = S + G * k_q
    for g in range(w.n_kv_heads):
        old = {bits(Kc_old[0, g, r]).tobytes() + bits(Vc_old[0, g, r]).tobytes() for r in range(win, w.L)}
        new = {bits(Kc2[0, g, r]).tobytes() + bits(Vc2[0, g, r]).tobytes() for r in range(win, w.L)}
        assert old == new

    # decoding goes on from the refreshed cache
    step = 0
    for t in range(T, T + 4):
        d = synth.make_decode_inputs(w, 0, t, dev)
        out = sk.decode_attn(d["q"], d["k_new"], d["v_new"], layer2)
        torch.cuda.synchronize()
        ref, _, step = O.decode_step(bits(d["q"][0]), bits(d["k_new"][0]), bits(d["v_new"][0]), Kc_ref, Vc_ref, step,
                                     S, k_q, R)
        err = np.abs(out[0].float().cpu().numpy() - ref)
        assert np.all(err <= 1e-2 + 1e-2 * np.abs(ref)), float(err.max())
    sk.close()
