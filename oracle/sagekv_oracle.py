"""Plain CPU oracle for the SAGE-KV hot path (arXiv 2503.08879, Section 2).

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement
of what the four steps compute.  It is imported by the tests, by the smoke
check and by the benchmark's CPU-baseline leg, and by nothing else; the CUDA
library never calls it and shares no code, tables or helpers with it.

Everything is numpy in float64.  bf16 tensors arrive as uint16 bit patterns and
are widened exactly (a bf16 is the top half of an fp32).  One call handles one
batch element and one layer.  Nothing here is blocked, fused or reordered
beyond what the definitions below say.

Notation (Section 2, Step 1, and Appendix A.2):
  N    context length, the last token included
  S    sink / initial tokens          (n_init)
  R    recent tokens                  (n_recent)
  E    eviction-region length,  E = N - 1 - S - R
  H_q, H_kv   query / key-value head counts,  G = H_q / H_kv
  k    tokens each query head keeps   (k_q in the C interface)
  L    reduced-cache length per KV head,  L = S + G*k + R + 1

Positions are 0-based here: sink [0,S), eviction region [S,S+E), recent window
[S+E, N-1), last token N-1  (the paper's P_{1:S}, P_{S+1:S+E}, P_{S+E+1:N-1}, P_N).

Section 3.1's baselines that are restated here for the comparison paths: StreamLLM_R
(rope_rotate, compact_window_rope: Appendix A.1) and the pooled reading of
Step 2 (select_pooled, compact_pooled, decode_step_pooled), and a Quest-style block-wise
per-step selection (quest_*), the comparison system of Section 3.1.

Pins (tests/test_oracle_pins.py): budget_split <- the numbers Appendix A.2
prints; score <- closed forms (uniform keys, one planted key), row sums, a
library softmax; select <- exhaustive subset search on tiny rows, library
argmax / top-k on distinct values; compact <- row-by-row source identity;
decode_step <- library scaled-dot-product attention for k = E, masked full
attention for any k, sink+recent attention for k = 0, ring contents after
t appends.  What is NOT pinned: that this heuristic reproduces the paper's
LongBench accuracy ("parity unpinned" for the method as a whole: it needs
the benchmark data and trained weights, neither of which is available).
"""

from __future__ import annotations

import numpy as np

__all__ = [
    "bf16_bits_to_f64",
    "f64_to_bf16_bits",
    "budget_split",
    "partition",
    "score",
    "select",
    "compact",
    "decode_step",
    "full_attention",
    "rope_rotate",
    "compact_window_rope",
    "select_pooled",
    "compact_pooled",
    "decode_step_pooled",
    "quest_summaries",
    "quest_bounds",
    "quest_select",
    "quest_attention",
]


# --------------------------------------------------------------------------
# bf16 <-> float64 (storage format only; no arithmetic of the method)
# --------------------------------------------------------------------------

def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even narrowing of finite float64 values to bf16 bits."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    rounded = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return (rounded >> np.uint64(16)).astype(np.uint16)


# --------------------------------------------------------------------------
# Appendix A.2: how a token budget B is divided
# --------------------------------------------------------------------------

def budget_split(B: int, G: int) -> tuple[int, int, int]:
    """(sink, k, recent) for token budget B and query-group number G.

    Appendix A.2: sink window B/4, k = B/(2G), recent window B/4.  When 2G
    does not divide B the appendix's own Qwen example (G = 7, B = 8192) takes
    k = 512 and gives every slot that is left to the recent window
    (8192 - 2048 - 7*512 = 2560).  Reading used here for the non-divisible
    case: k is the largest power of two not above B/(2G); the recent window is
    always B - sink - G*k.  In the divisible case this is the plain rule.
    """
    if B < 4 or G < 1:
        raise ValueError("budget_split needs B >= 4 and G >= 1")
    sink = B // 4
    if B % (2 * G) == 0:
        k = B // (2 * G)
    else:
        k = 1
        while 2 * k * 2 * G <= B:
            k *= 2
    recent = B - sink - G * k
    return sink, k, recent


# --------------------------------------------------------------------------
# Step 1: partition of the full cache
# --------------------------------------------------------------------------

def partition(N: int, S: int, R: int) -> dict:
    """Index ranges of the four parts (Step 1).  Half-open, 0-based."""
    E = N - 1 - S - R
    if S < 0 or R < 0 or E < 0:
        raise ValueError("need S >= 0, R >= 0 and S + R + 1 <= N")
    return {
        "E": E,
        "sink": (0, S),
        "evict": (S, S + E),
        "recent": (S + E, N - 1),
        "last": N - 1,
    }


# --------------------------------------------------------------------------
# Step 2a: attention scores of the last token over the eviction region
# --------------------------------------------------------------------------

def score(q_last_bits: np.ndarray, K_bits: np.ndarray, S: int, R: int,
          scale: float | None = None) -> np.ndarray:
    """Softmax attention of the last token's query over the evicted tokens.

    q_last_bits [H_q, d] and K_bits [H_kv, N, d] are bf16 bit patterns.  Query
    head h reads KV head h // G.  Returns p [H_q, E] in float64 with
        s[h, i] = scale * sum_c q[h, c] * K[h // G, S + i, c]
        p[h, i] = exp(s[h, i] - max_j s[h, j]) / sum_j exp(s[h, j] - max_j s[h, j])
    where j runs over the eviction region only (Step 2; scale = 1/sqrt(d)).
    """
    q = bf16_bits_to_f64(q_last_bits)
    H_q, d = q.shape
    H_kv, N, d2 = K_bits.shape
    assert d == d2 and H_q % H_kv == 0
    G = H_q // H_kv
    part = partition(N, S, R)
    E = part["E"]
    lo, hi = part["evict"]
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    p = np.zeros((H_q, E), dtype=np.float64)
    if E == 0:
        return p
    for g in range(H_kv):
        Kev = bf16_bits_to_f64(K_bits[g, lo:hi])          # [E, d]
        for j in range(G):
            h = g * G + j
            s = (Kev @ q[h]) * scale                      # [E]
            m = np.max(s)
            e = np.exp(s - m)
            p[h] = e / np.sum(e)
    return p


# --------------------------------------------------------------------------
# Step 2b: per-head top-k
# --------------------------------------------------------------------------

def select(p: np.ndarray, k: int, S: int) -> np.ndarray:
    """Top-k of every score row, the lower position winning a tie.

    p [H_q, E] in any float dtype; comparisons are made in that dtype.  Each
    row is ordered by (score descending, position ascending); the first
    min(k, E) entries are kept and re-ordered by position ascending (the
    reduced cache keeps token order, Appendix A.2).  Returns absolute token
    positions, int32 [H_q, min(k, E)], each in [S, S+E).
    """
    H_q, E = p.shape
    kk = min(int(k), E)
    out = np.zeros((H_q, kk), dtype=np.int32)
    pos = np.arange(E)
    for h in range(H_q):
        order = np.lexsort((pos, -p[h]))      # last key is the primary one
        out[h] = np.sort(order[:kk]) + S
    return out


# --------------------------------------------------------------------------
# Step 3: reduced cache C = Concat(S, E_topk, R, P_N)
# --------------------------------------------------------------------------

def compact(K_bits: np.ndarray, V_bits: np.ndarray, idx: np.ndarray,
            S: int, R: int) -> tuple[np.ndarray, np.ndarray]:
    """Reduced cache per KV head (Step 3).

    idx [H_q, k] are absolute positions chosen per query head.  "This yields
    H_q groups of the top-k" (Step 2) and the budget counts G*k selected slots
    per KV head (Appendix A.2), so the G lists of a KV head's query heads are
    laid side by side, duplicates kept:
        rows(g) = [0..S) ++ idx[g*G] ++ ... ++ idx[g*G+G-1] ++ [S+E..N-1) ++ [N-1]
    Returns (Kc, Vc) uint16 [H_kv, L, d] with L = S + G*k + R + 1; pure copies.
    """
    H_kv, N, d = K_bits.shape
    H_q, k = idx.shape
    G = H_q // H_kv
    E = partition(N, S, R)["E"]
    L = S + G * k + R + 1
    Kc = np.zeros((H_kv, L, d), dtype=np.uint16)
    Vc = np.zeros((H_kv, L, d), dtype=np.uint16)
    for g in range(H_kv):
        rows = list(range(0, S))
        for j in range(G):
            rows.extend(int(t) for t in idx[g * G + j])
        rows.extend(range(S + E, N - 1))
        rows.append(N - 1)
        assert len(rows) == L
        for r, t in enumerate(rows):
            Kc[g, r] = K_bits[g, t]
            Vc[g, r] = V_bits[g, t]
    return Kc, Vc


# --------------------------------------------------------------------------
# Plain softmax attention (the FullAttention baseline of Section 3.1)
# --------------------------------------------------------------------------

def full_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray,
                   keep: np.ndarray | None = None,
                   scale: float | None = None) -> tuple[np.ndarray, np.ndarray]:
    """softmax(q K^T * scale) V for grouped heads, float64 in and out.

    q [H_q, d]; K, V [H_kv, n, d]; keep [H_q, n] bool (False = logit -inf).
    Returns (o [H_q, d], lse [H_q]) with lse the log of the softmax denominator.
    """
    H_q, d = q.shape
    H_kv, n, _ = K.shape
    G = H_q // H_kv
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    o = np.zeros((H_q, d), dtype=np.float64)
    lse = np.full((H_q,), -np.inf, dtype=np.float64)
    for h in range(H_q):
        g = h // G
        s = (K[g] @ q[h]) * scale
        if keep is not None:
            s = np.where(keep[h], s, -np.inf)
        m = np.max(s)
        if not np.isfinite(m):
            continue
        e = np.exp(s - m)
        z = np.sum(e)
        o[h] = (e / z) @ V[g]
        lse[h] = m + np.log(z)
    return o, lse


# --------------------------------------------------------------------------
# Step 4: one decode step on the reduced cache
# --------------------------------------------------------------------------

def decode_step(q_bits: np.ndarray, k_new_bits, v_new_bits,
                Kc: np.ndarray, Vc: np.ndarray, step: int,
                S: int, k: int, R: int,
                scale: float | None = None) -> tuple[np.ndarray, np.ndarray, int]:
    """Append one token to the recent window, then attend (Step 4).

    The reduced cache of a KV head is [sink S | G segments of k | window R+1],
    the window being the R recent tokens followed by the last token, oldest
    first.  Appending token number `step` (0, 1, ...) overwrites window slot
    step mod (R+1): the oldest entry leaves, the size stays (Step 4).  With
    k_new_bits None nothing is appended.  Query head h = g*G + j then attends
    to the sink, to ITS OWN segment j and to the window, i.e. to S + k + R + 1
    entries, the length Step 3 states.  Kc, Vc are updated in place.
    Returns (o [H_q, d] float64, lse [H_q], step after the call).
    """
    H_kv, L, d = Kc.shape
    H_q = q_bits.shape[0]
    G = H_q // H_kv
    assert L == S + G * k + R + 1
    if k_new_bits is not None:
        slot = S + G * k + (step % (R + 1))
        for g in range(H_kv):
            Kc[g, slot] = k_new_bits[g]
            Vc[g, slot] = v_new_bits[g]
        step = step + 1
    keep = np.zeros((H_q, L), dtype=bool)
    for h in range(H_q):
        j = h % G
        keep[h, 0:S] = True
        keep[h, S + j * k: S + (j + 1) * k] = True
        keep[h, S + G * k: L] = True
    o, lse = full_attention(bf16_bits_to_f64(q_bits), bf16_bits_to_f64(Kc),
                            bf16_bits_to_f64(Vc), keep=keep, scale=scale)
    return o, lse, step


# --------------------------------------------------------------------------
# StreamLLM_R (Section 3.1 "Baselines", Appendix A.1): pre-RoPE cache, positions
# counted inside the window
# --------------------------------------------------------------------------

def rope_rotate(x: np.ndarray, pos, theta: float = 10000.0) -> np.ndarray:
    """Rotary position embedding of rows x [..., d] (float64) at positions pos.

    Dimension i < d/2 is paired with dimension i + d/2 (the layout of the
    Llama and Qwen models the paper runs); the pair is turned by the angle
    pos * theta**(-2i/d):
        y[i]       = x[i] cos(a_i) - x[i + d/2] sin(a_i)
        y[i + d/2] = x[i + d/2] cos(a_i) + x[i] sin(a_i),   a_i = pos * theta**(-2i/d)
    pos is a scalar or an array broadcastable to x's leading dimensions.
    """
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    half = d // 2
    inv_freq = float(theta) ** (-(np.arange(half, dtype=np.float64) * 2.0) / d)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c, s_ = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s_, x2 * c + x1 * s_], axis=-1)


def compact_window_rope(K_pre_bits: np.ndarray, V_bits: np.ndarray, S: int, R: int,
                        theta: float = 10000.0) -> tuple[np.ndarray, np.ndarray]:
    """StreamLLM_R's cache: sink + recent + last token of a PRE-RoPE key cache,
    every kept key rotated by its index inside the kept window (Appendix A.1:
    relative positions are assigned within the sliding window), values copied.

    K_pre_bits, V_bits uint16 [H_kv, N, d].  Returns (Kc, Vc) uint16
    [H_kv, S + R + 1, d]; row r of Kc is rope_rotate(K_pre[token(r)], r) rounded
    to bf16, with token(r) = r for r < S and N - 1 - (S + R) + r otherwise.
    """
    H_kv, N, d = K_pre_bits.shape
    E = partition(N, S, R)["E"]
    L = S + R + 1
    rows = list(range(0, S)) + list(range(S + E, N))
    assert len(rows) == L
    Kc = np.zeros((H_kv, L, d), dtype=np.uint16)
    Vc = np.zeros((H_kv, L, d), dtype=np.uint16)
    for g in range(H_kv):
        for r, t in enumerate(rows):
            Kc[g, r] = f64_to_bf16_bits(rope_rotate(bf16_bits_to_f64(K_pre_bits[g, t]), float(r), theta))
            Vc[g, r] = V_bits[g, t]
    return Kc, Vc


# --------------------------------------------------------------------------
# The pooled reading of Step 2 (one selection per KV head from the summed
# scores of its G query heads); the per-head reading above is the one the
# paper's budget rule fixes, this one is kept as the alternative
# --------------------------------------------------------------------------

def select_pooled(p: np.ndarray, K_sel: int, S: int, G: int) -> np.ndarray:
    """One top-K_sel per KV head from the sum of its G query heads' score rows.

    p [H_q, E]; rows g*G .. g*G+G-1 are added in float64, in head order, and
    rounded to p's dtype before they are compared (so a float32 caller compares
    float32 sums); then `select` on the H_kv summed rows.  Returns int32
    [H_kv, min(K_sel, E)].
    """
    H_q, E = p.shape
    H_kv = H_q // G
    pooled = np.zeros((H_kv, E), dtype=np.float64)
    for g in range(H_kv):
        for j in range(G):
            pooled[g] += p[g * G + j].astype(np.float64)
    return select(pooled.astype(p.dtype), K_sel, S)


def compact_pooled(K_bits: np.ndarray, V_bits: np.ndarray, idx: np.ndarray,
                   S: int, R: int) -> tuple[np.ndarray, np.ndarray]:
    """Reduced cache for the pooled reading: rows(g) = sink ++ idx[g] ++ recent ++ last."""
    H_kv = K_bits.shape[0]
    assert idx.shape[0] == H_kv
    return compact(K_bits, V_bits, idx, S, R)      # with H_q = H_kv the segment layout is one list per KV head


def decode_step_pooled(q_bits: np.ndarray, k_new_bits, v_new_bits, Kc: np.ndarray, Vc: np.ndarray,
                       step: int, S: int, K_sel: int, R: int,
                       scale: float | None = None) -> tuple[np.ndarray, np.ndarray, int]:
    """Step 4 for the pooled reading: every query head attends to ALL rows of its KV head's reduced cache."""
    H_kv, L, d = Kc.shape
    assert L == S + K_sel + R + 1
    if k_new_bits is not None:
        slot = S + K_sel + (step % (R + 1))
        for g in range(H_kv):
            Kc[g, slot] = k_new_bits[g]
            Vc[g, slot] = v_new_bits[g]
        step = step + 1
    o, lse = full_attention(bf16_bits_to_f64(q_bits), bf16_bits_to_f64(Kc), bf16_bits_to_f64(Vc), keep=None, scale=scale)
    return o, lse, step


# --------------------------------------------------------------------------
# Quest-style comparator (Section 3.1 "Baselines": a block-wise top-k selection
# method, run at every decode step on the FULL cache)
# --------------------------------------------------------------------------

def quest_summaries(K_bits: np.ndarray, S: int, R: int, block: int = 16) -> tuple[np.ndarray, np.ndarray]:
    """Element-wise minimum and maximum of the keys of every block of `block`
    consecutive tokens of the eviction region [S, S+E) (the last block may be
    shorter).  K_bits uint16 [H_kv, N, d].  Returns (kmin, kmax) as bf16 bit
    patterns [H_kv, n_blocks, d], n_blocks = ceil(E / block); minima and maxima
    of bf16 values are bf16 values, so nothing is rounded.
    """
    H_kv, N, d = K_bits.shape
    part = partition(N, S, R)
    E = part["E"]
    n_blocks = (E + block - 1) // block
    kmin = np.zeros((H_kv, n_blocks, d), dtype=np.uint16)
    kmax = np.zeros((H_kv, n_blocks, d), dtype=np.uint16)
    for g in range(H_kv):
        for j in range(n_blocks):
            lo, hi = S + j * block, min(S + E, S + (j + 1) * block)
            x = bf16_bits_to_f64(K_bits[g, lo:hi])
            kmin[g, j] = f64_to_bf16_bits(x.min(axis=0))
            kmax[g, j] = f64_to_bf16_bits(x.max(axis=0))
    return kmin, kmax


def quest_bounds(q_bits: np.ndarray, kmin_bits: np.ndarray, kmax_bits: np.ndarray,
                 scale: float | None = None) -> np.ndarray:
    """Upper bound of the attention logit of any token of a block:
        u[h, j] = scale * sum_c max(q[h, c] * kmin[h // G, j, c], q[h, c] * kmax[h // G, j, c])
    float64 [H_q, n_blocks]."""
    q = bf16_bits_to_f64(q_bits)
    H_q, d = q.shape
    H_kv, n_blocks, _ = kmin_bits.shape
    G = H_q // H_kv
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    lo, hi = bf16_bits_to_f64(kmin_bits), bf16_bits_to_f64(kmax_bits)
    u = np.zeros((H_q, n_blocks), dtype=np.float64)
    for h in range(H_q):
        g = h // G
        u[h] = np.sum(np.maximum(q[h] * lo[g], q[h] * hi[g]), axis=-1) * scale
    return u


def quest_select(u: np.ndarray, n_keep: int) -> np.ndarray:
    """The n_keep blocks of largest bound per query head (ties: lower block), ascending.  int32 [H_q, min(n_keep, n_blocks)]."""
    return select(u, n_keep, 0)


def quest_attention(q_bits: np.ndarray, K_bits: np.ndarray, V_bits: np.ndarray, blocks: np.ndarray,
                    S: int, R: int, block: int = 16, scale: float | None = None) -> np.ndarray:
    """Attention of every query head over sink + the tokens of its selected blocks + recent window + last token of
    the full cache.  float64 [H_q, d]."""
    H_kv, N, d = K_bits.shape
    H_q = q_bits.shape[0]
    E = partition(N, S, R)["E"]
    keep = np.zeros((H_q, N), dtype=bool)
    keep[:, :S] = True
    keep[:, S + E:] = True
    for h in range(H_q):
        for j in blocks[h]:
            keep[h, S + int(j) * block: min(S + E, S + (int(j) + 1) * block)] = True
    o, _ = full_attention(bf16_bits_to_f64(q_bits), bf16_bits_to_f64(K_bits), bf16_bits_to_f64(V_bits), keep=keep, scale=scale)
    return o
