"""Seeded random cases for select + compact: shapes, budgets, score distributions (skewed, few distinct values,
contiguous runs, signed, softmax-like) and what lies behind the rows (nothing, the true histogram of the group
maxima, that of other scores, noise).  Every case must give the oracle's indices and a bit-exact reduced cache."""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2503_08879_b200 import binding
    return binding


def score_keys(x):
    """Order-preserving 32-bit keys of float32 values (the kernels' comparison key)."""
    u = (np.asarray(x, dtype=np.float32) + np.float32(0.0)).view(np.uint32)
    return np.where(u & np.uint32(0x80000000), ~u, u | np.uint32(0x80000000)).astype(np.uint32)


def hint_of(rows, E):
    """What sagekv_score leaves behind rows of E scores: per row the 512-bin histogram of the maxima of the
    8 x 512 groups (16 bins per octave below the row maximum) and the four tag words, as uint32 [H, 516]."""
    H = rows.shape[0]
    chunk = ((E + 7) // 8 + 3) // 4 * 4
    out = np.zeros((H, 516), dtype=np.uint32)
    for h in range(H):
        gm = []
        for r in range(8):
            sl = rows[h, r * chunk:min(E, (r + 1) * chunk)]
            n_vec = len(sl) // 4
            g = np.full(512, -np.inf, dtype=np.float32)
            if n_vec:
                v = sl[:n_vec * 4].reshape(n_vec, 4).max(axis=1)
                pad = (-n_vec) % 512
                g = np.concatenate([v, np.full(pad, -np.inf, np.float32)]).reshape(-1, 512).max(axis=0)
            for t in range(len(sl) - n_vec * 4):
                g[t] = max(g[t], sl[n_vec * 4 + t])
            gm.append(g)
        gm = np.concatenate(gm)
        gm = gm[gm > -np.inf]
        kmax = int(score_keys(rows[h, :E].max()))
        bin0 = (kmax >> 19) - 511
        bins = np.clip((score_keys(gm) >> 19).astype(np.int64) - bin0, 0, 511)
        out[h, :512] = np.bincount(bins, minlength=512).astype(np.uint32)
        out[h, 512:] = [0x53414745, E, bin0, kmax]
    return out


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
        # behind the rows: 0 nothing, 1 the true histogram of the group maxima, 2 that of other scores, 3 noise
        mode = int(rng.integers(0, 4)) if E >= B.SKETCH_MIN_E else 0
        stride = E4 + (B.SKETCH_ROOM if mode else int(rng.integers(0, 3)) * 4)
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
