"""Seeded random cases for select + compact: shapes, budgets, score distributions (skewed, few distinct values,
contiguous runs, signed, softmax-like) and what lies behind the rows (nothing, the true group maxima, the maxima
of other scores, noise).  Every case must give the oracle's indices and a bit-exact reduced cache."""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2503_08879_b200 import binding
    return binding


def sketch_of(rows, E):
    H = rows.shape[0]
    chunk = ((E + 7) // 8 + 3) // 4 * 4
    sk = np.full((H, 8, 512), -np.inf, dtype=np.float32)
    for h in range(H):
        for r in range(8):
            sl = rows[h, r * chunk:min(E, (r + 1) * chunk)]
            n_vec = len(sl) // 4
            if n_vec:
                v = sl[:n_vec * 4].reshape(n_vec, 4).max(axis=1)
                pad = (-n_vec) % 512
                vv = np.concatenate([v, np.full(pad, -np.inf, np.float32)]).reshape(-1, 512).max(axis=0)
                sk[h, r] = vv
            for t in range(len(sl) - n_vec * 4):
                sk[h, r, t] = max(sk[h, r, t], sl[n_vec * 4 + t])
    return sk.reshape(H, 4096)

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


def bits(t):
    return t.detach().cpu().contiguous().view(torch.uint16).numpy()


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
        # behind the rows: 0 nothing, 1 the true group maxima, 2 those of other scores, 3 noise
        mode = int(rng.integers(0, 4)) if E >= B.SKETCH_MIN_E else 0
        stride = E4 + (B.SKETCH_ROOM if mode else int(rng.integers(0, 3)) * 4)
        buf = torch.zeros(H, stride, dtype=torch.float32, device="cuda")
        buf[:, :E] = torch.from_numpy(rows).cuda()
        if mode:
            if mode == 1:
                sk = sketch_of(rows, E)
            elif mode == 2:
                sk = sketch_of(gen_rows(rng, H, E, int(rng.integers(0, 5))), E)
            else:
                sk = (rng.standard_normal((H, 4096)) * 10.0 ** float(rng.integers(-6, 6))).astype(np.float32)
            buf[:, E4:E4 + 4096] = torch.from_numpy(sk).cuda()
            tag = np.array([0x53414745, E], dtype=np.int32).view(np.float32)
            buf[:, E4 + 4096:E4 + 4098] = torch.from_numpy(tag).cuda()
        N = S + E + R + 1
        K = torch.randn(1, Hkv, N, 128, generator=gen, device="cuda").to(torch.bfloat16)
        V = torch.randn(1, Hkv, N, 128, generator=gen, device="cuda").to(torch.bfloat16)
        sk_ = B.SageKV(H, Hkv, 128, 1, max_ctx=N, max_len=S + G * k_q + R + 1)
        layer = sk_.select_compact(buf, K, V, S, R, G * k_q)
        torch.cuda.synchronize()
        what = dict(case=case, G=G, Hkv=Hkv, E=E, k_q=k_q, S=S, R=R, kind=kind, behind=mode)
        idx = layer.indices()[0].cpu().numpy()
        assert np.array_equal(idx, O.select(rows, k_q, S)), what
        Kc_ref, Vc_ref = O.compact(bits(K[0]), bits(V[0]), idx, S, R)
        Kc, Vc = layer.cache()
        assert np.array_equal(bits(Kc[0]), Kc_ref) and np.array_equal(bits(Vc[0]), Vc_ref), what
        sk_.close()
