"""Pins for the CPU oracle: every function is checked against something other
than itself -- numbers the paper prints, closed forms, exhaustive search on tiny
inputs, or a library routine for the special case that reduces to one."""

import collections
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(x):
    """float array -> bf16 bit patterns via torch (independent of the oracle's own rounding)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.uint16).numpy().copy()


def bf16_val(bits):
    return torch.from_numpy(np.asarray(bits, dtype=np.uint16).copy()).view(torch.bfloat16).double().numpy()


def rand_bits(rng, *shape):
    return bf16(rng.standard_normal(shape))


# ---------------------------------------------------------------- bf16 helpers

def test_bf16_roundtrip_matches_torch():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(4096) * np.exp(rng.uniform(-20, 20, 4096))
    bits = bf16(x)
    assert np.array_equal(O.bf16_bits_to_f64(bits), bf16_val(bits))
    assert np.array_equal(O.f64_to_bf16_bits(x.astype(np.float32).astype(np.float64)), bits)
    # ties to even: 1 + 2^-8 is exactly half way between 1 and 1 + 2^-7
    assert O.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    assert O.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82


# ---------------------------------------------------------------- Appendix A.2

def test_budget_split_paper_numbers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "budget_split.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 2
    for B, G, sink, k, recent in (map(int, r) for r in rows):
        assert O.budget_split(B, G) == (sink, k, recent)
        assert sink + G * k + recent == B


@pytest.mark.parametrize("B,G", [(512, 4), (1024, 4), (2048, 7), (4096, 7), (2048, 1), (1000, 3)])
def test_budget_split_adds_up(B, G):
    sink, k, recent = O.budget_split(B, G)
    assert sink == B // 4 and sink + G * k + recent == B
    assert k <= B / (2 * G) and recent >= B // 4


# ---------------------------------------------------------------- Step 1

def test_partition_covers_disjointly():
    for N, S, R in [(12, 2, 3), (4096, 4, 64), (6, 4, 1), (5, 2, 2), (1, 0, 0)]:
        p = O.partition(N, S, R)
        cover = list(range(*p["sink"])) + list(range(*p["evict"])) + list(range(*p["recent"])) + [p["last"]]
        assert cover == list(range(N))
        assert p["E"] == N - 1 - S - R and p["recent"][1] - p["recent"][0] == R
    with pytest.raises(ValueError):
        O.partition(4, 2, 2)


# ---------------------------------------------------------------- Step 2a: score

def test_score_uniform_keys_gives_one_over_E():
    rng = np.random.default_rng(1)
    H_q, H_kv, d, N, S, R = 4, 2, 16, 40, 3, 5
    E = N - 1 - S - R
    K = rand_bits(rng, H_kv, N, d)
    K[:, S:S + E] = K[:, S:S + 1]                # every evictable key the same
    p = O.score(rand_bits(rng, H_q, d), K, S, R)
    assert p.shape == (H_q, E)
    np.testing.assert_allclose(p, 1.0 / E, rtol=1e-12)


def test_score_one_planted_key_closed_form():
    # q = 2*e_0, planted key 3*e_0 at eviction offset i0, all other keys 0:
    # logit 6/sqrt(d) there and 0 elsewhere => p = e^x / (e^x + E - 1).
    H_q, H_kv, d, N, S, R = 2, 1, 64, 30, 4, 6
    E = N - 1 - S - R
    q = np.zeros((H_q, d)); q[:, 0] = 2.0
    q[1, 0] = -2.0                                # sign of the logit matters
    K = np.zeros((H_kv, N, d))
    i0 = 7
    K[0, S + i0, 0] = 3.0
    # decoys outside the eviction region must change nothing
    K[0, 0, 0] = 100.0; K[0, S + E, 0] = 100.0; K[0, N - 1, 0] = 100.0; K[0, S - 1, 0] = 100.0
    p = O.score(bf16(q), bf16(K), S, R)
    x = 6.0 / math.sqrt(d)
    want0 = math.exp(x) / (math.exp(x) + E - 1)
    want1 = math.exp(-x) / (math.exp(-x) + E - 1)
    assert abs(p[0, i0] - want0) < 1e-14 and abs(p[1, i0] - want1) < 1e-14
    np.testing.assert_allclose(np.delete(p[0], i0), (1 - want0) / (E - 1), rtol=1e-12)
    # explicit scale overrides 1/sqrt(d)
    p2 = O.score(bf16(q), bf16(K), S, R, scale=0.5)
    assert abs(p2[0, i0] - math.exp(3.0) / (math.exp(3.0) + E - 1)) < 1e-14


def test_score_query_head_reads_its_kv_head():
    # KV head g has one strong key at eviction offset 2+g; all queries equal.
    H_q, H_kv, d, N, S, R = 6, 3, 8, 20, 2, 2
    q = np.zeros((H_q, d)); q[:, 1] = 4.0
    K = np.zeros((H_kv, N, d))
    for g in range(H_kv):
        K[g, S + 2 + g, 1] = 5.0
    p = O.score(bf16(q), bf16(K), S, R)
    assert [int(np.argmax(p[h])) for h in range(H_q)] == [2, 2, 3, 3, 4, 4]


def test_score_rows_sum_to_one_and_match_library_softmax():
    rng = np.random.default_rng(2)
    H_q, H_kv, d, N, S, R = 8, 2, 128, 300, 4, 16
    E = N - 1 - S - R
    qb, Kb = rand_bits(rng, H_q, d), rand_bits(rng, H_kv, N, d)
    p = O.score(qb, Kb, S, R)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, atol=1e-12)
    qt = torch.from_numpy(bf16_val(qb)); Kt = torch.from_numpy(bf16_val(Kb))
    Kt = Kt.repeat_interleave(H_q // H_kv, dim=0)[:, S:S + E]
    want = torch.softmax(torch.einsum("hd,hnd->hn", qt, Kt) / math.sqrt(d), dim=-1).numpy()
    np.testing.assert_allclose(p, want, rtol=1e-10)


def test_score_brute_force_python_loops():
    rng = np.random.default_rng(3)
    H_q, H_kv, d, N, S, R = 4, 2, 8, 11, 2, 3
    E = N - 1 - S - R
    qb, Kb = rand_bits(rng, H_q, d), rand_bits(rng, H_kv, N, d)
    p = O.score(qb, Kb, S, R)
    qv, Kv = bf16_val(qb), bf16_val(Kb)
    for h in range(H_q):
        g = h // (H_q // H_kv)
        logits = [math.fsum(qv[h, c] * Kv[g, S + i, c] for c in range(d)) / math.sqrt(d) for i in range(E)]
        z = math.fsum(math.exp(s) for s in logits)
        for i in range(E):
            assert abs(p[h, i] - math.exp(logits[i]) / z) < 1e-13


def test_score_empty_region():
    rng = np.random.default_rng(4)
    p = O.score(rand_bits(rng, 2, 8), rand_bits(rng, 1, 6, 8), 2, 3)
    assert p.shape == (2, 0)


# ---------------------------------------------------------------- Step 2b: select

def _exhaustive_topk(row, k):
    """Among all k-subsets: the largest exact sum, then the lexicographically
    smallest sorted position tuple (= lower positions win ties)."""
    best = None
    for sub in itertools.combinations(range(len(row)), k):
        key = (-sum(int(row[i]) for i in sub), sub)
        if best is None or key < best:
            best = key
    return list(best[1])


def test_select_exhaustive_small_rows_with_ties():
    rng = np.random.default_rng(5)
    for trial in range(60):
        E = int(rng.integers(1, 10))
        k = int(rng.integers(0, E + 1))
        row = rng.integers(0, 4, size=E)          # small integers: many ties, exact sums
        S = int(rng.integers(0, 5))
        for dtype in (np.float32, np.float64):
            got = O.select(row[None, :].astype(dtype), k, S)
            assert got.dtype == np.int32 and got.shape == (1, k)
            assert [int(t) - S for t in got[0]] == _exhaustive_topk(row, k)


def test_select_special_cases():
    rng = np.random.default_rng(6)
    p = rng.random((5, 200)).astype(np.float32)
    p[3, 17] = p[3, 150] = 2.0                    # tied maxima: first one wins
    one = O.select(p, 1, 9)
    assert [int(t) for t in one[:, 0]] == [int(np.argmax(p[h])) + 9 for h in range(5)]
    assert int(one[3, 0]) == 17 + 9
    full = O.select(p, 200, 9)
    assert np.array_equal(full, np.tile(np.arange(9, 209, dtype=np.int32), (5, 1)))
    clamp = O.select(p, 1000, 9)                  # k above E is clamped to E
    assert np.array_equal(clamp, full)
    flat = O.select(np.full((2, 50), 0.02, dtype=np.float32), 7, 3)
    assert np.array_equal(flat, np.tile(np.arange(3, 10, dtype=np.int32), (2, 1)))
    assert O.select(p, 0, 9).shape == (5, 0)


def test_select_matches_library_topk_on_distinct_values():
    rng = np.random.default_rng(7)
    p = rng.permutation(5000).reshape(5, 1000).astype(np.float32)
    got = O.select(p, 37, 4)
    want = torch.topk(torch.from_numpy(p), 37, dim=1).indices.numpy()
    for h in range(5):
        assert list(got[h]) == sorted(int(i) + 4 for i in want[h])
        assert np.all(np.diff(got[h]) > 0)


# ---------------------------------------------------------------- Step 3: compact

def test_compact_hand_worked_layout():
    # N=12, S=2, R=3 => E=6 (positions 2..7), recent 8..10, last 11; G=2, k=2.
    H_kv, N, d, S, R = 2, 12, 4, 2, 3
    K = np.zeros((H_kv, N, d), dtype=np.uint16)
    V = np.zeros((H_kv, N, d), dtype=np.uint16)
    for g in range(H_kv):
        for t in range(N):
            K[g, t] = 1000 * (g + 1) + 10 * t + np.arange(d)
            V[g, t] = 30000 + 1000 * (g + 1) + 10 * t + np.arange(d)
    idx = np.array([[3, 6], [2, 3], [5, 7], [4, 5]], dtype=np.int32)   # heads 0,1 -> kv 0; 2,3 -> kv 1
    Kc, Vc = O.compact(K, V, idx, S, R)
    want_rows = {0: [0, 1, 3, 6, 2, 3, 8, 9, 10, 11], 1: [0, 1, 5, 7, 4, 5, 8, 9, 10, 11]}
    assert Kc.shape == Vc.shape == (H_kv, 2 + 2 * 2 + 3 + 1, d)
    for g in range(H_kv):
        for r, t in enumerate(want_rows[g]):
            assert np.array_equal(Kc[g, r], K[g, t]) and np.array_equal(Vc[g, r], V[g, t])


# ---------------------------------------------------------------- Step 4: decode

def _sdpa(q, K, V, G, mask=None):
    """Library attention in float64.  q [H_q,d]; K,V [H_kv,n,d]; mask [H_q,n] bool."""
    qt = torch.from_numpy(q)[None, :, None, :]
    Kt = torch.from_numpy(K).repeat_interleave(G, dim=0)[None]
    Vt = torch.from_numpy(V).repeat_interleave(G, dim=0)[None]
    m = None if mask is None else torch.from_numpy(mask)[None, :, None, :]
    return torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt, attn_mask=m)[0, :, 0].numpy()


def _pipeline(rng, H_q, H_kv, d, N, S, R, k):
    qb, Kb, Vb = rand_bits(rng, H_q, d), rand_bits(rng, H_kv, N, d), rand_bits(rng, H_kv, N, d)
    p = O.score(qb, Kb, S, R)
    idx = O.select(p.astype(np.float32), k, S)
    Kc, Vc = O.compact(Kb, Vb, idx, S, R)
    return qb, Kb, Vb, idx, Kc, Vc


def test_decode_k_equals_E_is_full_attention():
    rng = np.random.default_rng(8)
    H_q, H_kv, d, N, S, R = 6, 2, 32, 90, 3, 7
    E = N - 1 - S - R
    qb, Kb, Vb, idx, Kc, Vc = _pipeline(rng, H_q, H_kv, d, N, S, R, E)
    o, lse, step = O.decode_step(qb, None, None, Kc, Vc, 0, S, E, R)
    assert step == 0
    want = _sdpa(bf16_val(qb), bf16_val(Kb), bf16_val(Vb), H_q // H_kv)
    np.testing.assert_allclose(o, want, rtol=1e-10, atol=1e-12)
    logits = np.einsum("hd,hnd->hn", bf16_val(qb), np.repeat(bf16_val(Kb), H_q // H_kv, axis=0)) / math.sqrt(d)
    np.testing.assert_allclose(lse, torch.logsumexp(torch.from_numpy(logits), dim=1).numpy(), rtol=1e-12)


@pytest.mark.parametrize("k", [0, 1, 5, 19])
def test_decode_equals_masked_full_attention(k):
    rng = np.random.default_rng(9 + k)
    H_q, H_kv, d, N, S, R = 8, 2, 16, 70, 2, 6
    E = N - 1 - S - R
    G = H_q // H_kv
    qb, Kb, Vb, idx, Kc, Vc = _pipeline(rng, H_q, H_kv, d, N, S, R, k)
    q2 = rand_bits(rng, H_q, d)                   # any query, not only the last token's
    o, _, _ = O.decode_step(q2, None, None, Kc, Vc, 0, S, k, R)
    mask = np.zeros((H_q, N), dtype=bool)
    mask[:, :S] = True; mask[:, S + E:] = True
    for h in range(H_q):
        mask[h, idx[h]] = True
    assert mask.sum(axis=1).tolist() == [S + k + R + 1] * H_q      # the length Step 3 states
    want = _sdpa(bf16_val(q2), bf16_val(Kb), bf16_val(Vb), G, mask)
    np.testing.assert_allclose(o, want, rtol=1e-10, atol=1e-12)
    if k == 0:                                    # sink + recent only (StreamLLM with absolute positions)
        keep = list(range(S)) + list(range(S + E, N))
        want0 = _sdpa(bf16_val(q2), bf16_val(Kb)[:, keep], bf16_val(Vb)[:, keep], G)
        np.testing.assert_allclose(o, want0, rtol=1e-10, atol=1e-12)


def test_decode_recent_window_rolls():
    rng = np.random.default_rng(20)
    H_q, H_kv, d, N, S, R, k = 4, 2, 16, 40, 2, 3, 4
    G = H_q // H_kv
    qb, Kb, Vb, idx, Kc, Vc = _pipeline(rng, H_q, H_kv, d, N, S, R, k)
    L = Kc.shape[1]
    E = N - 1 - S - R
    # model of the window: the R recent tokens and the last token, oldest first
    win = [collections.deque(((Kb[g, t].copy(), Vb[g, t].copy()) for t in range(S + E, N)), maxlen=R + 1)
           for g in range(H_kv)]
    step = 0
    for t in range(2 * (R + 1) + 3):
        q = rand_bits(rng, H_q, d); kn = rand_bits(rng, H_kv, d); vn = rand_bits(rng, H_kv, d)
        o, _, step = O.decode_step(q, kn, vn, Kc, Vc, step, S, k, R)
        assert step == t + 1 and Kc.shape[1] == L
        for g in range(H_kv):
            win[g].append((kn[g].copy(), vn[g].copy()))      # deque drops the oldest
        for h in range(H_q):
            g, j = h // G, h % G
            rowsK = [Kb[g, i] for i in range(S)] + [Kb[g, i] for i in idx[h]] + [kv[0] for kv in win[g]]
            rowsV = [Vb[g, i] for i in range(S)] + [Vb[g, i] for i in idx[h]] + [kv[1] for kv in win[g]]
            want = _sdpa(bf16_val(q[h:h + 1]), bf16_val(np.stack(rowsK))[None], bf16_val(np.stack(rowsV))[None], 1)
            np.testing.assert_allclose(o[h], want[0], rtol=1e-10, atol=1e-12)
        if t + 1 >= R + 1:                        # window now holds only appended tokens
            for g in range(H_kv):
                got = {Kc[g, r].tobytes() for r in range(S + G * k, L)}
                assert got == {kv[0].tobytes() for kv in win[g]}


# ---------------------------------------------------------------- StreamLLM_R: rotary positions inside the window

def test_rope_rotation_group_properties():
    """Rotation by 0 is the identity, rotations add up, norms are kept, and the product of a rotated query and
    a rotated key depends only on the difference of their positions (what makes positions 'relative')."""
    rng = np.random.default_rng(41)
    x, y = rng.standard_normal((5, 128)), rng.standard_normal((5, 128))
    assert np.array_equal(O.rope_rotate(x, 0.0), x)
    np.testing.assert_allclose(O.rope_rotate(O.rope_rotate(x, 3.0), 11.0), O.rope_rotate(x, 14.0), atol=1e-12)
    np.testing.assert_allclose(np.linalg.norm(O.rope_rotate(x, 977.0), axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    for p, q in ((7, 2), (1007, 1002), (40000, 39995)):
        a = np.sum(O.rope_rotate(x, float(p)) * O.rope_rotate(y, float(q)), axis=-1)
        b = np.sum(O.rope_rotate(x, 5.0) * y, axis=-1)
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-9)
    np.testing.assert_allclose(O.rope_rotate(x, np.arange(5.0))[3], O.rope_rotate(x[3], 3.0), atol=1e-14)


def test_rope_is_a_complex_multiplication():
    """The textbook form: (x_i + i x_{i+d/2}) * exp(i * pos * theta^(-2i/d)); a swapped sign, a wrong pairing
    (neighbouring dimensions) or a wrong exponent fails this."""
    rng = np.random.default_rng(42)
    d, theta, pos = 64, 500000.0, 1234.0
    x = rng.standard_normal(d)
    z = (x[: d // 2] + 1j * x[d // 2:]) * np.exp(1j * pos * theta ** (-np.arange(d // 2) * 2.0 / d))
    np.testing.assert_allclose(O.rope_rotate(x, pos, theta), np.concatenate([z.real, z.imag]), atol=1e-12)


def test_rope_matches_the_llama_implementation_of_a_library():
    tr = pytest.importorskip("transformers")
    from transformers.models.llama.modeling_llama import LlamaRotaryEmbedding, apply_rotary_pos_emb
    cfg = tr.LlamaConfig(hidden_size=4 * 32, num_attention_heads=4, head_dim=32, rope_theta=10000.0,
                         max_position_embeddings=256)
    rot = LlamaRotaryEmbedding(cfg)
    rng = np.random.default_rng(43)
    x = rng.standard_normal((1, 1, 9, 32)).astype(np.float32)          # [batch, heads, positions, head_dim]
    pos = torch.arange(20, 29)[None]
    cos, sin = rot(torch.from_numpy(x), pos)
    got, _ = apply_rotary_pos_emb(torch.from_numpy(x), torch.from_numpy(x), cos, sin)
    want = O.rope_rotate(x[0, 0].astype(np.float64), np.arange(20.0, 29.0), 10000.0)
    np.testing.assert_allclose(got[0, 0].double().numpy(), want, atol=2e-5)


def test_compact_window_rope_rows_and_positions():
    """Which token lands in which row, rotated by the row's own index; values untouched."""
    rng = np.random.default_rng(44)
    H, N, d, S, R = 2, 40, 16, 3, 5
    K, V = rand_bits(rng, H, N, d), rand_bits(rng, H, N, d)
    Kc, Vc = O.compact_window_rope(K, V, S, R, theta=100.0)
    tokens = [0, 1, 2, 34, 35, 36, 37, 38, 39]
    assert Kc.shape == (H, 9, d)
    for r, t in enumerate(tokens):
        assert np.array_equal(Vc[:, r], V[:, t])
        x = bf16_val(K[:, t])
        z = (x[:, : d // 2] + 1j * x[:, d // 2:]) * np.exp(1j * r * 100.0 ** (-np.arange(d // 2) * 2.0 / d))
        assert np.array_equal(Kc[:, r], bf16(np.concatenate([z.real, z.imag], axis=-1)))
    assert np.array_equal(Kc[:, 0], K[:, 0])                              # position 0: no rotation


# ---------------------------------------------------------------- the pooled reading of Step 2

def test_select_pooled_is_select_on_the_summed_rows():
    rng = np.random.default_rng(45)
    p = rng.random((6, 50)).astype(np.float32)
    idx = O.select_pooled(p, 7, 4, G=3)
    assert idx.shape == (2, 7)
    for g in range(2):
        summed = (p[3 * g].astype(np.float64) + p[3 * g + 1] + p[3 * g + 2]).astype(np.float32)
        best = sorted(sorted(range(50), key=lambda i: (-summed[i], i))[:7])
        assert idx[g].tolist() == [4 + i for i in best]
    assert np.array_equal(O.select_pooled(p, 7, 4, G=1), O.select(p, 7, 4))   # G = 1: nothing to pool


def test_decode_pooled_equals_full_attention_over_the_kept_rows():
    rng = np.random.default_rng(46)
    Hq, Hkv, N, d, S, R, Ksel = 4, 2, 60, 16, 2, 6, 9
    K, V, q = rand_bits(rng, Hkv, N, d), rand_bits(rng, Hkv, N, d), rand_bits(rng, Hq, d)
    p = O.score(q, K, S, R).astype(np.float32)
    idx = O.select_pooled(p, Ksel, S, G=2)
    Kc, Vc = O.compact_pooled(K, V, idx, S, R)
    o, lse, step = O.decode_step_pooled(q, None, None, Kc, Vc, 0, S, Ksel, R)
    for h in range(Hq):
        g = h // 2
        rows = list(range(S)) + idx[g].tolist() + list(range(N - 1 - R, N))
        want = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(bf16_val(q[h]))[None, None], torch.from_numpy(bf16_val(K[g, rows]))[None],
            torch.from_numpy(bf16_val(V[g, rows]))[None])[0, 0]
        np.testing.assert_allclose(o[h], want.numpy(), atol=1e-10)
    assert step == 0


# ---------------------------------------------------------------- Quest-style block selection

def test_quest_bound_dominates_every_token_and_is_tight_for_single_token_blocks():
    rng = np.random.default_rng(51)
    Hq, Hkv, N, d, S, R = 4, 2, 133, 16, 3, 6
    K, q = rand_bits(rng, Hkv, N, d), rand_bits(rng, Hq, d)
    E = N - 1 - S - R
    kmin, kmax = O.quest_summaries(K, S, R, block=16)
    assert kmin.shape == (Hkv, (E + 15) // 16, d)
    u = O.quest_bounds(q, kmin, kmax)
    logits = np.einsum("hc,htc->ht", bf16_val(q), bf16_val(K)[np.repeat(np.arange(Hkv), 2)]) / math.sqrt(d)
    for h in range(Hq):
        for j in range(u.shape[1]):
            blk = logits[h, S + 16 * j: min(S + E, S + 16 * (j + 1))]
            assert np.all(blk <= u[h, j] + 1e-12)
    # the summaries themselves, block by block, from torch's own bf16 arithmetic
    kv = torch.from_numpy(bf16_val(K))
    assert np.array_equal(bf16_val(kmin[1, 2]), kv[1, S + 32: S + 48].min(dim=0).values.numpy())
    assert np.array_equal(bf16_val(kmax[0, -1]), kv[0, S + 16 * (u.shape[1] - 1): S + E].max(dim=0).values.numpy())
    # blocks of one token: the bound is the logit itself
    kmin1, kmax1 = O.quest_summaries(K, S, R, block=1)
    np.testing.assert_allclose(O.quest_bounds(q, kmin1, kmax1), logits[:, S:S + E], atol=1e-12)


def test_quest_attention_is_masked_full_attention():
    rng = np.random.default_rng(52)
    Hq, Hkv, N, d, S, R = 4, 2, 90, 16, 2, 5
    K, V, q = rand_bits(rng, Hkv, N, d), rand_bits(rng, Hkv, N, d), rand_bits(rng, Hq, d)
    kmin, kmax = O.quest_summaries(K, S, R)
    blocks = O.quest_select(O.quest_bounds(q, kmin, kmax), 2)
    assert blocks.shape == (Hq, 2) and np.all(np.diff(blocks, axis=1) > 0)
    o = O.quest_attention(q, K, V, blocks, S, R)
    E = N - 1 - S - R
    for h in range(Hq):
        g = h // 2
        rows = list(range(S)) + [t for j in blocks[h] for t in range(S + 16 * j, min(S + E, S + 16 * (j + 1)))] + list(range(S + E, N))
        want = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(bf16_val(q[h]))[None, None], torch.from_numpy(bf16_val(K[g, rows]))[None],
            torch.from_numpy(bf16_val(V[g, rows]))[None])[0, 0]
        np.testing.assert_allclose(o[h], want.numpy(), atol=1e-10)
