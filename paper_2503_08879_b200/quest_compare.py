"""SAGE-KV's one-shot selection beside a Quest-style per-step block selection, on the same synthetic caches.

Section 3.2 of the paper compares the two by task accuracy at a token budget (its "memory efficiency").  Neither
the tasks nor the models are available here, so this is a synthetic analogue and says so: the caches carry planted
heavy tokens (keys aligned with the last token's query), and what is reported, at an equal token budget per query
head, is
  - recall: the share of a head's planted tokens that the selection keeps (of those the budget could hold),
  - bytes a decode step has to read per layer: SAGE-KV reads its reduced cache; the block method reads the block
    summaries of the whole eviction region and then the rows of the blocks it picked, for every query head,
  - microseconds per layer-step of the selection work a decode step needs (none for SAGE-KV: it selected once).
The block method re-selects with every new query, which helps when later queries look elsewhere; the synthetic
queries here do not drift, so that advantage does not show.  Run:  python -m paper_2503_08879_b200.quest_compare
"""

from __future__ import annotations

import sys

import torch

from . import binding as B
from . import synth


def run(name: str, device="cuda:0", reps: int = 20) -> dict:
    w = synth.workload(name).with_(n_layers=1)
    dev = torch.device(device)
    lay = synth.make_layer(w, 0, dev)
    S, R, E, G = w.n_init, w.n_recent, w.E, w.G
    nb = (E + 15) // 16
    keep = max(1, w.k_q // 16)
    sk = B.SageKV(w.n_q_heads, w.n_kv_heads, w.head_dim, w.batch, max_ctx=w.n_ctx, max_len=w.L, device=dev)
    scores = sk.score(lay["q_last"], lay["K"], S, R)
    layer = sk.select_compact(scores, lay["K"], lay["V"], S, R, w.n_sel)
    kmin = torch.empty(w.batch, w.n_kv_heads, nb, 128, dtype=torch.bfloat16, device=dev)
    kmax = torch.empty_like(kmin)
    stride = (nb + 3) // 4 * 4
    u = torch.empty(w.batch * w.n_q_heads, stride, dtype=torch.float32, device=dev)
    blocks = torch.empty(w.batch * w.n_q_heads, keep, dtype=torch.int32, device=dev)
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))

    def per_step():
        B.sagekv_quest_bounds(sk.ctx, lay["q_last"], kmin, kmax, nb, u, stride)
        B.sagekv_select_topk(sk.ctx, u, stride, nb, keep, blocks)

    B.sagekv_quest_build(sk.ctx, lay["K"], w.n_ctx, S, R, kmin, kmax)
    per_step()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        B.sagekv_quest_build(sk.ctx, lay["K"], w.n_ctx, S, R, kmin, kmax)
    e1.record()
    for _ in range(reps):
        per_step()
    e2.record()
    torch.cuda.synchronize()
    build_us, step_us = e0.elapsed_time(e1) * 1e3 / reps, e1.elapsed_time(e2) * 1e3 / reps

    idx = layer.indices().cpu()                       # [B, H_q, k_q] token positions
    blk = blocks.view(w.batch, w.n_q_heads, keep).cpu()
    rec_sage, rec_quest, n_heads = 0.0, 0.0, 0
    for b in range(w.batch):
        for h in range(w.n_q_heads):
            g, j = divmod(h, G)
            pos = lay["heavy"][b][g].cpu()
            mine = pos[torch.arange(pos.numel()) % G == j]           # planted token number t belongs to head g*G + t % G
            if mine.numel() == 0:
                continue
            can = min(mine.numel(), w.k_q)
            kept = torch.isin(mine, idx[b, h].long()).sum().item()
            in_blocks = torch.isin((mine - S) // 16, blk[b, h].long()).sum().item()
            rec_sage += kept / can
            rec_quest += min(in_blocks, can) / can
            n_heads += 1
    row = 2 * w.head_dim * 2                                          # bytes of a token's K and V rows
    sage_bytes = w.batch * w.n_kv_heads * w.L * row
    quest_bytes = (w.batch * w.n_kv_heads * nb * w.head_dim * 2 * 2
                   + w.batch * w.n_q_heads * (S + keep * 16 + R + 1) * row)
    sk.close()
    return {"workload": name, "tokens_per_head": w.k_q, "blocks_per_head": keep, "recall_sagekv": rec_sage / n_heads,
            "recall_blocks": rec_quest / n_heads, "bytes_per_layer_step_sagekv": sage_bytes,
            "bytes_per_layer_step_blocks": quest_bytes, "summary_build_us_per_layer": build_us,
            "block_selection_us_per_layer_step": step_us,
            "summary_build_gbs": w.batch * w.n_kv_heads * E * 256 / (build_us * 1e-6) / 1e9}


def main(argv):
    names = argv or ["C1", "C2", "C3-2048"]
    print("| workload | tokens / head | recall SAGE-KV | recall blocks (x16) | MB per layer-step SAGE-KV | MB blocks | "
          "summaries us/layer (GB/s) | block selection us/layer-step |")
    print("|---|---|---|---|---|---|---|---|")
    for n in names:
        r = run(n)
        print("| %s | %d | %.3f | %.3f | %.2f | %.2f | %.1f (%.0f) | %.1f |" % (
            r["workload"], r["tokens_per_head"], r["recall_sagekv"], r["recall_blocks"], r["bytes_per_layer_step_sagekv"] / 1e6,
            r["bytes_per_layer_step_blocks"] / 1e6, r["summary_build_us_per_layer"], r["summary_build_gbs"],
            r["block_selection_us_per_layer_step"]))


if __name__ == "__main__":
    main(sys.argv[1:])
