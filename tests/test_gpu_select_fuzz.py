"""Seeded random cases for select + compact: shapes, budgets, score distributions (skewed, few distinct values,
contiguous runs, signed, softmax-like) and what lies behind the rows (nothing, the true histogram of the group
maxima, that of other scores, noise).  Every case must give the oracle's indices and a bit-exact reduced cache."""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O
from helpers import HINT_MIN_E, HINT_WORDS, bits, hint_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2503_08879_b200 import binding
    return binding


def gen_rows(rng, H, E, kind):
    if kind == 0: r = rng.random((H, E), dtype=np.float32) ** rng.integers(1, 12)
    elif kind == 1: r = (rng.integers(0, rng.integers(2, 200), (H, E)) / 64.0).astype(np.float32)
    elif kind == 2:
        r = (rng.random((H, E), dtype=np.float32) * 1e-3).astype(np.float32)
        for h in range(H):
            for _ in range(rng.integers(1, 9)):
                a = rng.integers(0, E); L = rng.integers(1, 2000)
                r[h, a:a + L] += rng.random(min(L, E - a), dtype=np.float32)
    elif kind == 3: r = rng.standard_normal((H, E)).astype(np.float32)
    else:
        r = np.exp(rng.standard_normal((H, E)) * 3).astype(np.float32); r /= r.sum(axis=1, keepdims=True)
    return np.ascontiguousarray(r.astype(np.float32))


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_random_cases_match_the_oracle(B, seed):
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    for case in range(16):
        G = int(rng.choice([1, 2, 4, 7, 8])); Hkv = int(rng.integers(1, 3)); H = G * Hkv
        E = int(rng.choice([rng.integers(1, 3000), rng.integers(3000, 40000), rng.integers(40000, 200000)]))
        k_q = int(min(E, rng.choice([rng.integers(1, 64), rng.integers(64, 1200), rng.integers(1200, 5000)])))
        S, R = int(rng.integers(0, 6)), int(rng.integers(0, 40))
        kind = int(rng.integers(0, 5))
        rows = gen_rows(rng, H, E, kind)
        E4 = (E + 3) // 4 * 4
        # behind the rows: 0 nothing, 1 the true histogram of the group maxima, 2 that of other scores, 3 noise
        mode = int(rng.integers(0, 4)) if E >= HINT_MIN_E else 0
        N = S + E + R + 1
        sk_ = B.SageKV(H, Hkv, 128, 1, max_ctx=N, max_len=S + G * k_q + R + 1)
        if mode:
            sk_.set_select_hint(1)
            stride = sk_.score_stride(N, S, R)
            assert stride >= E4 + HINT_WORDS
        else:                                                   # hint off: any stride, whatever lies behind the rows
            stride = E4 + int(rng.choice([0, 4, 8, HINT_WORDS + 4]))
        buf = torch.zeros(H, stride, dtype=torch.float32, device="cuda")
        buf[:, :E] = torch.from_numpy(rows).cuda()
        if mode:
            if mode == 1:
                words = hint_of(rows, E)
            elif mode == 2:
                words = hint_of(gen_rows(rng, H, E, int(rng.integers(0, 5))), E)
            else:
                words = rng.integers(0, 2 ** 32, (H, 516), dtype=np.uint64).astype(np.uint32)
                words[:, 512:514] = [0x53414745, E]
            buf[:, E4:E4 + 516] = torch.from_numpy(words.view(np.float32)).cuda()
        elif stride >= E4 + HINT_WORDS:                         # words that claim to be a hint, and must not be read
            words = rng.integers(0, 2 ** 32, (H, HINT_WORDS), dtype=np.uint64).astype(np.uint32)
            words[:, 512:514] = [0x53414745, E]
            buf[:, E4:E4 + 516] = torch.from_numpy(words.view(np.float32)).cuda()
        K = torch.randn(1, Hkv, N, 128, generator=gen, device="cuda").to(torch.bfloat16)
        V = torch.randn(1, Hkv, N, 128, generator=gen, device="cuda").to(torch.bfloat16)
        layer = sk_.select_compact(buf, K, V, S, R, G * k_q)
        torch.cuda.synchronize()
        what = dict(case=case, G=G, Hkv=Hkv, E=E, k_q=k_q, S=S, R=R, kind=kind, behind=mode)
        idx = layer.indices()[0].cpu().numpy()
        assert np.array_equal(idx, O.select(rows, k_q, S)), what
        Kc_ref, Vc_ref = O.compact(bits(K[0]), bits(V[0]), idx, S, R)
        Kc, Vc = layer.cache()
        assert np.array_equal(bits(Kc[0]), Kc_ref) and np.array_equal(bits(Vc[0]), Vc_ref), what
        assert sk_.status() == 0, what
        sk_.close()
