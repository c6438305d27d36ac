"""Seeded random cases for the score step: batch, heads, group size, context and partition lengths, strided K,
and both row strides (with and without the room behind the rows).  Scores within the relative tolerance of the
oracle, rows summing to one, padding beyond the documented extras untouched."""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O
from helpers import HINT_MIN_E, HINT_WORDS, bits

pytestmark = pytest.mark.gpu
SCORE_RTOL = 1e-3


@pytest.fixture(scope="module")
def B():
    from paper_2503_08879_b200 import binding
    return binding


@pytest.mark.parametrize("seed", [301, 302])
def test_random_cases_match_the_oracle(B, seed):
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    for case in range(12):
        G = int(rng.choice([1, 2, 4, 7, 8])); Hkv = int(rng.choice([1, 2, 4])); H = G * Hkv
        Bt = int(rng.choice([1, 1, 2, 3]))
        S, R = int(rng.integers(0, 6)), int(rng.integers(0, 100))
        E = int(rng.choice([rng.integers(1, 600), rng.integers(600, 20000), rng.integers(20000, 60000)]))
        N = S + E + R + 1
        pad_tokens = int(rng.integers(0, 3)) * 8                 # K rows may be wider than 128 elements apart
        Kfull = torch.randn(Bt, Hkv, N, 128 + pad_tokens, generator=gen, device="cuda").to(torch.bfloat16)
        K = Kfull[..., :128]
        q = (torch.randn(Bt, H, 128, generator=gen, device="cuda") * float(rng.choice([0.5, 1.0, 4.0]))).to(torch.bfloat16)
        E4 = (E + 3) // 4 * 4
        wide = bool(rng.integers(0, 2)) and E >= HINT_MIN_E    # with the hint for the select step behind the rows
        scale = float(rng.choice([0.0, 0.0, 0.05, 0.2]))        # 0: the default 1/sqrt(d)
        sk = B.SageKV(H, Hkv, 128, Bt, max_ctx=N, max_len=64, softmax_scale=scale)
        if wide:
            sk.set_select_hint(1)
            stride = sk.score_stride(N, S, R) + int(rng.integers(0, 2)) * 8
        else:
            stride = E4 + int(rng.choice([0, 4, 8, HINT_WORDS + 8]))
        buf = torch.full((Bt * H, stride), 7.5, dtype=torch.float32, device="cuda")
        sk.score(q, K, S, R, scores=buf)
        torch.cuda.synchronize()
        what = dict(case=case, G=G, Hkv=Hkv, batch=Bt, S=S, R=R, E=E, wide=wide, k_row=128 + pad_tokens, scale=scale)
        got = buf.view(Bt, H, stride).cpu().numpy()
        for b in range(Bt):
            ref = O.score(bits(q[b]), bits(K[b].contiguous()), S, R, scale=scale if scale > 0 else None)
            np.testing.assert_allclose(got[b, :, :E].astype(np.float64), ref, rtol=SCORE_RTOL, atol=1e-30, err_msg=str(what))
            np.testing.assert_allclose(got[b, :, :E].astype(np.float64).sum(axis=1), 1.0, atol=1e-4, err_msg=str(what))
        if wide:
            assert (got[:, :, E4 + 516:] == 7.5).all() and (got[:, :, E:E4] == 7.5).all(), what
        else:
            assert (got[:, :, E:] == 7.5).all(), what
        assert sk.status() == 0, what
        sk.close()
