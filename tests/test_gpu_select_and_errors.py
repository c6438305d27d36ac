"""Select on hand-made score rows (ties, constants, negative values, guard bands) and the
argument-error matrix of the C interface.  Nothing here relies on the score kernel."""

import ctypes

import numpy as np
import pytest
import torch

from oracle import sagekv_oracle as O
from helpers import HINT_WORDS, bits, hint_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2503_08879_b200 import binding
    return binding


def run_select(B, rows: np.ndarray, k_q: int, S=3, R=5, H_kv=None, pad=8):
    """rows [H_q, E] fp32 -> (idx [H_q, k_q], Kc, Vc, K, V) with random K/V and guard bands checked."""
    H_q, E = rows.shape
    H_kv = H_kv or H_q
    G = H_q // H_kv
    N = S + E + R + 1
    g = torch.Generator(device="cuda").manual_seed(1234 + E)
    K = torch.randn(1, H_kv, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    V = torch.randn(1, H_kv, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    stride = (E + 3) // 4 * 4 + pad
    buf = torch.full((H_q, stride), 7.5, dtype=torch.float32, device="cuda")
    buf[:, :E] = torch.from_numpy(rows).cuda()
    sk = B.SageKV(H_q, H_kv, 128, 1, max_ctx=N, max_len=S + G * k_q + R + 1)
    layer = sk.new_layer(S, R, G * k_q)
    canary = 0x5A5A
    layer.Kc.view(torch.int16).fill_(canary)
    layer.Vc.view(torch.int16).fill_(canary)
    layer.idx.fill_(-77)
    before = buf.clone()
    sk.select_compact(buf, K, V, S, R, G * k_q, layer)
    torch.cuda.synchronize()
    assert torch.equal(before, buf)                       # scores are read-only, padding untouched
    kk = min(k_q, E)
    idx = layer.indices()[0].cpu().numpy()
    assert layer.idx.flatten()[H_q * kk:].eq(-77).all()   # nothing written past the used part
    Kc_ref, Vc_ref = O.compact(bits(K[0]), bits(V[0]), idx, S, R)
    Kc, Vc = layer.cache()
    assert np.array_equal(bits(Kc[0]), Kc_ref) and np.array_equal(bits(Vc[0]), Vc_ref)
    sk.close()
    return idx


@pytest.mark.parametrize("E,k_q", [(1, 1), (5, 2), (33, 33), (600, 7), (2049, 100), (5000, 64), (16385, 479),
                                   (40000, 1000), (70001, 1983)])
def test_select_random_rows_bit_exact(B, E, k_q):
    rng = np.random.default_rng(E)
    rows = rng.random((4, E), dtype=np.float32) ** 8       # skewed like softmax rows
    idx = run_select(B, rows, k_q, H_kv=2)
    assert np.array_equal(idx, O.select(rows, k_q, 3))


@pytest.mark.parametrize("E", [200000, 524027])
@pytest.mark.parametrize("k_q", [959, 1983])
def test_select_long_rows_several_load_rounds(B, E, k_q):
    """Rows long enough that a thread of the prefilter goes through its slice in several rounds of eight vectors:
    staged slices at E = 200000 (two rounds), unstaged ones at E = 524027 (four), each with a run of large scores
    across a slice border and a group of equal scores at the cut."""
    rng = np.random.default_rng(E + k_q)
    rows = (rng.random((2, E), dtype=np.float32) ** 10).astype(np.float32)
    slice_len = ((E + 7) // 8 + 3) // 4 * 4
    for h in range(2):
        rows[h, slice_len * 2 - 100: slice_len * 2 + 140] = 0.97 + 0.02 * rng.random(240, dtype=np.float32)   # a run over a border
        kth = np.sort(rows[h])[::-1][k_q - 1]
        tie = rng.choice(E, 60, replace=False)
        rows[h, tie] = kth                                                                                  # equal scores at the cut
    idx = run_select(B, rows, k_q, H_kv=1)
    assert np.array_equal(idx, O.select(rows, k_q, 3))


def test_select_ties_lowest_position_wins(B):
    E = 9000
    rng = np.random.default_rng(5)
    rows = np.empty((6, E), dtype=np.float32)
    rows[0] = 0.25                                          # every score equal
    rows[1] = rng.integers(0, 3, E)                         # three distinct values
    rows[2] = rng.integers(0, 50, E) / 64.0
    rows[3] = np.where(rng.random(E) < 0.01, 1.0, 0.5)      # few large, threshold inside a huge tie
    rows[4] = rng.standard_normal(E)                        # negative values order correctly
    rows[5] = -np.abs(rng.standard_normal(E)); rows[5, ::7] = -0.0; rows[5, 3::7] = 0.0
    for k_q in (1, 17, 300, 4500, 9000):
        idx = run_select(B, rows, k_q, H_kv=3)
        assert np.array_equal(idx, O.select(rows, k_q, 3))


@pytest.mark.parametrize("k_q,winners,ties", [(300, 280, 40), (500, 300, 420), (600, 400, 700)])
def test_select_tie_group_straddles_the_cut_in_the_prefilter_path(B, k_q, winners, ties):
    """Few enough equal scores that the prefilter path is taken, placed so that the k-th score lies inside
    the group: exactly the lowest positions of the group must be kept.  The three sizes end in the exact
    ranking of a small group, of one that takes several rounds, and in the hand-over to the general path."""
    E = 60000
    rng = np.random.default_rng(11)
    rows = (rng.random((4, E), dtype=np.float32) * 0.5).astype(np.float32)
    for h in range(4):
        top = rng.choice(E, winners, replace=False)           # clear winners
        rows[h, top] = 0.9 + 0.05 * rng.random(winners, dtype=np.float32)
        rest = np.setdiff1d(np.arange(E), top)
        tie = rng.choice(rest, ties, replace=False)           # equal scores: k_q - winners of them make the cut
        rows[h, tie] = 0.75
    idx = run_select(B, rows, k_q, H_kv=2)
    want = O.select(rows, k_q, 3)
    assert np.array_equal(idx, want)
    for h in range(4):
        tie_pos = np.sort(np.nonzero(rows[h] == np.float32(0.75))[0]) + 3
        kept = np.intersect1d(idx[h], tie_pos)
        assert np.array_equal(kept, tie_pos[:k_q - winners])


def test_select_large_scores_in_contiguous_runs(B):
    """Winners that sit next to each other (whole vectors and whole warps of hits) and a run that crosses the
    border between two CTAs' slices: the candidate lists must still come out in position order."""
    E, k_q = 60000, 500
    rng = np.random.default_rng(12)
    rows = (rng.random((4, E), dtype=np.float32) * 0.5).astype(np.float32)
    slice_len = (E + 7) // 8
    for h in range(4):
        for start in (1234 + 97 * h, slice_len * 3 - 70, 41000 + h):
            rows[h, start:start + 150] = 0.8 + 0.1 * rng.random(150, dtype=np.float32)
        rows[h, rng.choice(E, 100, replace=False)] += 0.6
    assert np.array_equal(run_select(B, rows, k_q, H_kv=2), O.select(rows, k_q, 3))


def test_cache_rows_read_from_pinned_host_memory(B):
    """K and V may stay in pinned host memory (addressable from the device): the gather then pulls only the
    kept rows over the bus.  Same indices and the same reduced cache as with device-resident K and V."""
    E, k_q, S, R = 20000, 200, 4, 16
    rows = np.random.default_rng(21).random((4, E), dtype=np.float32) ** 6
    N = S + E + R + 1
    g = torch.Generator(device="cuda").manual_seed(77)
    K = torch.randn(1, 2, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    V = torch.randn(1, 2, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    scores = torch.from_numpy(rows).cuda()
    sk = B.SageKV(4, 2, 128, 1, max_ctx=N, max_len=S + 2 * k_q + R + 1)
    on_device = sk.select_compact(scores, K, V, S, R, 2 * k_q)
    in_place = sk.select_compact(scores, K.cpu().pin_memory(), V.cpu().pin_memory(), S, R, 2 * k_q)
    torch.cuda.synchronize()
    assert torch.equal(on_device.indices(), in_place.indices())
    assert np.array_equal(on_device.indices()[0].cpu().numpy(), O.select(rows, k_q, S))
    for a, b in zip(on_device.cache(), in_place.cache()):
        assert torch.equal(a, b)
    sk.close()


@pytest.mark.parametrize("hint", ["true", "far too high", "far too low", "garbage", "wrong tag"])
def test_histogram_behind_the_rows_is_only_a_hint(B, hint):
    """The floats behind a long score row may hold the histogram of the row's group maxima (written by
    sagekv_score): whatever they hold, the selection is the oracle's.  A bound that is too low gives too many
    candidates, one that is too high too few; both send the row through the path that takes the maxima itself."""
    E, k_q, S, R = 60000, 300, 3, 5
    rng = np.random.default_rng(31)
    rows = (rng.random((4, E), dtype=np.float32) ** 6).astype(np.float32)
    E4 = (E + 3) // 4 * 4
    N = S + E + R + 1
    sk = B.SageKV(4, 2, 128, 1, max_ctx=N, max_len=S + 2 * k_q + R + 1)
    sk.set_select_hint(1)
    stride = sk.score_stride(N, S, R)
    assert stride >= E4 + HINT_WORDS
    buf = torch.zeros(4, stride, dtype=torch.float32, device="cuda")
    buf[:, :E] = torch.from_numpy(rows).cuda()
    words = hint_of(rows, E)
    if hint == "far too high":
        words[:, :512] = 0
        words[:, 511] = 4096                                  # every group maximum claimed to be near the row maximum
    elif hint == "far too low":
        words[:, 514] -= 40 * 16                              # bins laid 40 octaves lower: the bound lands far below
        words[:, 515] = words[:, 514] + 511 << 19
    elif hint == "garbage":
        words[:, :512] = rng.integers(0, 2 ** 32, (4, 512), dtype=np.uint64).astype(np.uint32)
        words[:, 514:] = rng.integers(0, 2 ** 32, (4, 2), dtype=np.uint64).astype(np.uint32)
    elif hint == "wrong tag":
        words[:, 513] += 1
    buf[:, E4:E4 + 516] = torch.from_numpy(words.view(np.float32)).cuda()
    g = torch.Generator(device="cuda").manual_seed(5)
    K = torch.randn(1, 2, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    V = torch.randn(1, 2, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    before = buf.clone()
    layer = sk.select_compact(buf, K, V, S, R, 2 * k_q)
    torch.cuda.synchronize()
    assert torch.equal(before.view(torch.int32), buf.view(torch.int32))      # read-only, hint included
    idx = layer.indices()[0].cpu().numpy()
    assert np.array_equal(idx, O.select(rows, k_q, S))
    Kc_ref, Vc_ref = O.compact(bits(K[0]), bits(V[0]), idx, S, R)
    Kc, Vc = layer.cache()
    assert np.array_equal(bits(Kc[0]), Kc_ref) and np.array_equal(bits(Vc[0]), Vc_ref)
    sk.close()


def test_score_leaves_the_histogram_when_the_rows_have_room(B):
    """sagekv_score with the wider row stride: scores as without it, and behind each row the histogram of the
    group maxima with its tag; the floats after those 516 words stay untouched."""
    Hq, Hkv, N, S, R = 4, 2, 20000, 4, 16
    E = N - 1 - S - R
    g = torch.Generator(device="cuda").manual_seed(9)
    q = torch.randn(1, Hq, 128, generator=g, device="cuda").to(torch.bfloat16)
    K = torch.randn(1, Hkv, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    sk = B.SageKV(Hq, Hkv, 128, 1, max_ctx=N, max_len=64)
    E4 = (E + 3) // 4 * 4
    narrow = torch.zeros(Hq, E4, dtype=torch.float32, device="cuda")
    assert sk.score_stride(N, S, R) == E4                        # hint off: no room asked for
    sk.score(q, K, S, R, scores=narrow)
    sk.set_select_hint(1)
    wide = torch.full((Hq, sk.score_stride(N, S, R) + 12), 7.5, dtype=torch.float32, device="cuda")
    for _ in range(2):                                           # the second call starts from the first one's counts
        sk.score(q, K, S, R, scores=wide)
    torch.cuda.synchronize()
    assert torch.equal(narrow[:, :E], wide[:, :E])
    got = wide[:, E4:E4 + 516].cpu().numpy().view(np.uint32)
    assert np.array_equal(got, hint_of(wide[:, :E].cpu().numpy(), E))
    assert (wide[:, E4 + 516:] == 7.5).all() and (wide[:, E:E4] == 7.5).all()
    sk.close()


def test_without_the_hint_nothing_behind_the_rows_is_touched_or_believed(B):
    """Hint off (the default): score rows may be interleaved with other data of the caller, e.g. one
    [rows, layers, E] tensor with a row stride of layers * E.  sagekv_score must leave the neighbouring data
    bit-exact, and sagekv_select_compact must not read it: here it holds words that look like a valid hint
    claiming every group maximum sits at the row maximum."""
    Hq, Hkv, N, S, R, k_q, layers = 4, 2, 20000, 4, 16, 200, 3
    E = N - 1 - S - R
    E4 = (E + 3) // 4 * 4
    g = torch.Generator(device="cuda").manual_seed(19)
    q = torch.randn(1, Hq, 128, generator=g, device="cuda").to(torch.bfloat16)
    K = torch.randn(1, Hkv, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    V = torch.randn(1, Hkv, N, 128, generator=g, device="cuda").to(torch.bfloat16)
    sk = B.SageKV(Hq, Hkv, 128, 1, max_ctx=N, max_len=S + 2 * k_q + R + 1)
    tensor = torch.full((Hq, layers, E4), 3.25, dtype=torch.float32, device="cuda")
    fake = np.zeros((Hq, HINT_WORDS), dtype=np.uint32)
    fake[:, 511] = 4096
    fake[:, 512:] = [0x53414745, E, 100, 0x7fffffff]
    tensor[:, 1, :HINT_WORDS] = torch.from_numpy(fake.view(np.float32)).cuda()      # right behind layer 0's rows
    before = tensor.clone()
    rows = tensor[:, 0, :]                                                          # row stride layers * E4
    B.sagekv_score(sk.ctx, q, K, N, S, R, rows, rows.stride(0))
    torch.cuda.synchronize()
    assert torch.equal(tensor[:, 1:].view(torch.int32), before[:, 1:].view(torch.int32))
    assert (tensor[:, 0, E:] == 3.25).all()
    layer = sk.new_layer(S, R, 2 * k_q)
    B.sagekv_select_compact(sk.ctx, rows, rows.stride(0), K, V, N, S, R, 2 * k_q, layer.idx, layer.Kc, layer.Vc,
                            layer.state)
    torch.cuda.synchronize()
    assert torch.equal(tensor[:, 1:].view(torch.int32), before[:, 1:].view(torch.int32))
    got = rows[:, :E].cpu().numpy()
    assert np.array_equal(layer.indices()[0].cpu().numpy(), O.select(got, k_q, S))
    assert sk.status() == 0
    sk.close()


def test_select_threshold_differs_only_in_low_bits(B):
    E = 20000
    base = np.float32(0.001)
    ulps = np.random.default_rng(6).integers(0, 40, (2, E)).astype(np.uint32)
    rows = (np.full((2, E), base, dtype=np.float32).view(np.uint32) + ulps).view(np.float32)
    for k_q in (5, 999):
        assert np.array_equal(run_select(B, rows, k_q), O.select(rows, k_q, 3))


def test_select_is_deterministic(B):
    rows = np.random.default_rng(8).random((4, 30000), dtype=np.float32)
    a = run_select(B, rows, 479, H_kv=1)
    b = run_select(B, rows, 479, H_kv=1)
    assert np.array_equal(a, b)


def test_argument_errors_are_reported_before_launch(B):
    lib, C = B.lib, ctypes
    sk = B.SageKV(8, 2, 128, 1, max_ctx=1000, max_len=200)
    K = torch.zeros(1, 2, 1000, 128, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(1, 8, 128, dtype=torch.bfloat16, device="cuda")
    sc = torch.zeros(8, 1000, dtype=torch.float32, device="cuda")
    layer = sk.new_layer(4, 16, 32)
    code = lambda f, *a: pytest.raises(B.SagekvError, f, *a).value.code
    # score
    assert code(B.sagekv_score, sk.ctx, None, K, 1000, 4, 16, sc, 1000) == B.ERR_INVALID
    assert code(B.sagekv_score, sk.ctx, q, K, 1000, 600, 400, sc, 1000) == B.ERR_INVALID      # S+R+1 > N
    assert code(B.sagekv_score, sk.ctx, q, K, 1000, -1, 16, sc, 1000) == B.ERR_INVALID
    assert code(B.sagekv_score, sk.ctx, q, K, 1000, 4, 16, sc, 500) == B.ERR_INVALID          # row stride < E
    assert code(B.sagekv_score, sk.ctx, q, K, 1000, 4, 16, sc, 998) == B.ERR_ALIGN            # stride % 4
    assert code(B.sagekv_score, sk.ctx, q, K, 2000, 4, 16, sc, 2000) == B.ERR_UNSUPPORTED     # beyond max_ctx
    assert code(B.sagekv_score, sk.ctx, q.view(-1)[4:].view(-1), K, 1000, 4, 16, sc, 1000) == B.ERR_ALIGN
    # select_compact
    sel = lambda **kw: B.sagekv_select_compact(sk.ctx, kw.get("sc", sc), kw.get("stride", 1000), K, K, 1000,
                                               kw.get("S", 4), kw.get("R", 16), kw.get("k", 32), layer.idx,
                                               layer.Kc, layer.Vc, layer.state)
    assert pytest.raises(B.SagekvError, sel, k=30).value.code == B.ERR_INVALID                # k % G != 0
    assert pytest.raises(B.SagekvError, sel, k=-4).value.code == B.ERR_INVALID
    assert pytest.raises(B.SagekvError, sel, S=990).value.code == B.ERR_INVALID
    assert pytest.raises(B.SagekvError, sel, k=400).value.code == B.ERR_UNSUPPORTED           # L > max_len
    assert pytest.raises(B.SagekvError, sel, sc=None).value.code == B.ERR_INVALID
    # decode
    sel()
    out = torch.empty_like(q)
    kn = torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda")
    assert code(B.sagekv_decode_attn, sk.ctx, q, kn, None, layer.Kc, layer.Vc, layer.state, out) == B.ERR_INVALID
    assert code(B.sagekv_decode_attn, sk.ctx, None, None, None, layer.Kc, layer.Vc, layer.state, out) == B.ERR_INVALID
    bad = B.CacheState(4, 8, 32, 16, 17, 99, layer.step.data_ptr())                           # len inconsistent
    assert code(B.sagekv_decode_attn, sk.ctx, q, None, None, layer.Kc, layer.Vc, bad, out) == B.ERR_INVALID
    B.sagekv_decode_attn(sk.ctx, q, None, None, layer.Kc, layer.Vc, layer.state, out)
    torch.cuda.synchronize()                                                                   # context still healthy
    # the mode setters take 0..2 (the group mode 0..1) and nothing else
    for setter in (lib.sagekv_set_overlap, lib.sagekv_set_select_overlap, lib.sagekv_set_decode_variant):
        assert setter(sk.ctx, 3) == B.ERR_INVALID and setter(sk.ctx, -1) == B.ERR_INVALID and setter(sk.ctx, 2) == 0 and setter(sk.ctx, 0) == 0
    assert lib.sagekv_set_group_mode(sk.ctx, 2) == B.ERR_INVALID
    # create
    h = C.c_void_p()
    shp = B.Shape(8, 2, 64, 1, 0.0)
    assert lib.sagekv_create(C.byref(h), C.byref(shp), 1000, 100) == B.ERR_UNSUPPORTED and not h.value
    shp = B.Shape(32, 2, 128, 1, 0.0)
    assert lib.sagekv_create(C.byref(h), C.byref(shp), 1000, 100) == B.ERR_UNSUPPORTED        # G = 16
    shp = B.Shape(8, 3, 128, 1, 0.0)
    assert lib.sagekv_create(C.byref(h), C.byref(shp), 1000, 100) == B.ERR_INVALID
    sk.close()
