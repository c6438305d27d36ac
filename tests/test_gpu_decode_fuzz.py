"""Seeded random cases for decode attention: batch, KV heads and group size (which decide the cluster size of the
launch), reduced-cache lengths from a few rows to several passes, window lengths, query scales.  The reduced cache
is built by select_compact from random scores and by the oracle from the same scores; a few decode steps must
agree within the output tolerance and leave bit-identical caches."""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O
from helpers import bits

pytestmark = pytest.mark.gpu
OUT_ATOL, OUT_RTOL = 1e-2, 1e-2


@pytest.fixture(scope="module")
def B():
    from paper_2503_08879_b200 import binding
    return binding


def f32(a):
    return (a.astype(np.uint32) << 16).view(np.float32)


@pytest.mark.parametrize("seed", [201, 202, 203])
def test_random_cases_match_the_oracle(B, seed):
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    for case in range(12):
        G = int(rng.choice([1, 2, 4, 7, 8])); Hkv = int(rng.choice([1, 2, 4, 8])); H = G * Hkv
        Bt = int(rng.choice([1, 1, 2, 3, 4, 6]))
        S, R = int(rng.integers(0, 6)), int(rng.integers(0, 200))
        L_target = int(rng.choice([rng.integers(2, 300), rng.integers(300, 2400), rng.integers(2400, 7000)]))
        k_q = max(0, (L_target - S - R - 1) // G)
        E = k_q + int(rng.integers(0, 50))
        if E == 0:
            k_q = 0
        N, L = S + E + R + 1, S + G * k_q + R + 1
        K = torch.randn(Bt, Hkv, N, 128, generator=gen, device="cuda").to(torch.bfloat16)
        V = torch.randn(Bt, Hkv, N, 128, generator=gen, device="cuda").to(torch.bfloat16)
        rows = rng.random((Bt * H, max(E, 1)), dtype=np.float32)
        buf = torch.zeros(Bt * H, max(4, (E + 3) // 4 * 4), dtype=torch.float32, device="cuda")
        if E:
            buf[:, :E] = torch.from_numpy(rows[:, :E]).cuda()
        sm_scale = float(rng.choice([0.0, 0.0, 0.05, 0.2]))      # softmax scale of the context; 0: the default 1/sqrt(d)
        sk = B.SageKV(H, Hkv, 128, Bt, max_ctx=N, max_len=L, softmax_scale=sm_scale)
        sk.set_overlap(int(rng.integers(0, 2)))
        sk.set_decode_variant(2 if case % 3 == 2 else 0)          # every third case on the tensor-memory kernel (where it applies)
        layer = sk.select_compact(buf if k_q else None, K, V, S, R, G * k_q)
        torch.cuda.synchronize()
        what = dict(case=case, G=G, Hkv=Hkv, batch=Bt, S=S, R=R, k_q=k_q, E=E, L=L, softmax_scale=sm_scale)
        caches = []
        for b in range(Bt):
            idx = O.select(rows[b * H:(b + 1) * H, :E], k_q, S) if k_q else np.zeros((H, 0), np.int32)
            caches.append(list(O.compact(bits(K[b]), bits(V[b]), idx, S, R)))
        steps = [0] * Bt
        for t in range(int(rng.integers(1, 4))):
            scale = float(rng.choice([0.3, 1.0, 3.0]))
            q = torch.randn(Bt, H, 128, generator=gen, device="cuda").to(torch.bfloat16) * scale
            kn = torch.randn(Bt, Hkv, 128, generator=gen, device="cuda").to(torch.bfloat16)
            vn = torch.randn(Bt, Hkv, 128, generator=gen, device="cuda").to(torch.bfloat16)
            out = sk.decode_attn(q, kn, vn, layer)
            torch.cuda.synchronize()
            for b in range(Bt):
                ref, _, steps[b] = O.decode_step(bits(q[b]), bits(kn[b]), bits(vn[b]), caches[b][0], caches[b][1],
                                                 steps[b], S, k_q, R, scale=sm_scale if sm_scale > 0 else None)
                got = f32(bits(out[b])).astype(np.float64)
                assert np.all(np.abs(got - ref) <= OUT_ATOL + OUT_RTOL * np.abs(ref)), what
        Kc, Vc = layer.cache()
        for b in range(Bt):
            assert np.array_equal(bits(Kc[b]), caches[b][0]) and np.array_equal(bits(Vc[b]), caches[b][1]), what
        assert sk.status() == 0, what
        sk.close()
