"""Helpers shared by the GPU tests: bit views, the kernels' comparison key, and the layout of the hint that
sagekv_score can leave behind the score rows (one copy, so that the tests cannot drift apart)."""

import numpy as np
import torch

HINT_WORDS = 516       # 512 histogram bins + four tag words behind a row (hint mode 1)
HINT_MIN_E = 14337     # shortest row for which the hint is written


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.uint16).numpy()


def score_keys(x):
    """Order-preserving 32-bit keys of float32 values (the kernels' comparison key)."""
    u = (np.asarray(x, dtype=np.float32) + np.float32(0.0)).view(np.uint32)
    return np.where(u & np.uint32(0x80000000), ~u, u | np.uint32(0x80000000)).astype(np.uint32)


def hint_of(rows, E):
    """What sagekv_score leaves behind rows of E scores in hint mode 1: per row the 512-bin histogram of the
    maxima of the 8 x 512 groups (16 bins per octave below the row maximum) and the four tag words, as
    uint32 [H, 516]."""
    H = rows.shape[0]
    chunk = ((E + 7) // 8 + 3) // 4 * 4
    out = np.zeros((H, HINT_WORDS), dtype=np.uint32)
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
