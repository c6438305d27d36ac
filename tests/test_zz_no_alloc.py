"""sagekv_score_static: the score step for callers that cannot allocate device memory (a serving
process whose cache manager already owns the GPU's memory cannot afford the cudaMalloc, or its
device-wide synchronisation, that creating a context costs).  The entry point keeps its scratch in a
fixed array inside the library, so its results must equal those of sagekv_score and lie within the score
tolerance of the CPU oracle, call after call, although every call reuses the same array.  Collected last on
purpose."""

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O
from helpers import bits
from paper_2503_08879_b200 import synth

pytestmark = pytest.mark.gpu

SCORE_RTOL = 1e-3     # the tolerance the score parity tests use


def test_static_score_matches_context_score_on_two_calls_in_a_row():
    from paper_2503_08879_b200 import binding as B
    dev = "cuda"
    # two different problems back to back: the second must not see anything of the first in the shared array
    cases = [synth.workload("C2").with_(n_ctx=20011, n_layers=1),
             synth.workload("C4-b1").with_(n_ctx=9000, batch=2, n_layers=1)]
    for w in cases:
        lay = synth.make_layer(w, 0, dev)
        sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L)
        want = sk.score(lay["q_last"], lay["K"], w.n_init, w.n_recent)
        got = torch.full_like(want, -1.0)
        shape = B.Shape(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, 0.0)
        before = torch.cuda.memory_allocated()
        B.sagekv_score_static(shape, lay["q_last"], lay["K"], w.n_ctx, w.n_init, w.n_recent, got, got.stride(0))
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        a, b = got[:, : w.E].cpu().numpy(), want[:, : w.E].cpu().numpy()
        np.testing.assert_allclose(a, b, rtol=SCORE_RTOL, atol=1e-30)
        np.testing.assert_allclose(a.sum(axis=1), 1.0, atol=1e-4)
        for bi in range(w.batch):                                # and against the oracle itself, not only the sibling call
            ref = O.score(bits(lay["q_last"][bi]), bits(lay["K"][bi]), w.n_init, w.n_recent)
            np.testing.assert_allclose(a.reshape(w.batch, w.n_q_heads, -1)[bi].astype(np.float64), ref,
                                       rtol=SCORE_RTOL, atol=1e-30)
        assert torch.equal(got[:, w.E:], torch.full_like(got[:, w.E:], -1.0))     # row padding untouched
        sk.close()


def test_static_score_rejects_problems_beyond_its_fixed_scratch():
    from paper_2503_08879_b200 import binding as B
    # 64 rows x 1024 chunks of 256 tokens = 65536 partial entries > 32768
    q = torch.zeros(2, 32, 128, dtype=torch.bfloat16, device="cuda")
    K = torch.zeros(1, 1, 8, 128, dtype=torch.bfloat16, device="cuda")     # never read: the call must refuse first
    scores = torch.zeros(4, dtype=torch.float32, device="cuda")
    shape = B.Shape(32, 8, 128, 2, 0.0)
    with pytest.raises(B.SagekvError) as e:
        B.sagekv_score_static(shape, q, K, 262144 + 133, 4, 128, scores, 262144)
    assert e.value.code == B.ERR_TOO_LARGE
    assert "fixed scratch" in str(e.value)
    bad = B.Shape(32, 8, 64, 1, 0.0)
    with pytest.raises(B.SagekvError) as e:
        B.sagekv_score_static(bad, q, K, 100, 4, 16, scores, 80)
    assert e.value.code == B.ERR_UNSUPPORTED
