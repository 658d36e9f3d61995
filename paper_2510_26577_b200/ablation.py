"""Breadth pruning, depth pruning and dynamic rerank switched on and off across batch sizes.

The paper's ablation (Sec. "Ablation study") shows that cost-aware sizing matters more as the batch
grows.  This script reproduces the *mechanism* on synthetic inputs: the Llama-3-8B-shaped batch sweep
with the synthetic cost tables of `workloads.cost_table_arrays` and peaked draft logits (values decay
slowly with depth, as those of a trained draft head do).  For every batch size and setting it prints
what the sizing decided (n_i per layer, layers generated, N) and what the step then costs on this
GPU (tree build, one layer of verification attention).  No accept lengths: those need real models.

  python -m paper_2510_26577_b200.ablation [--batches 1,4,16,64] [--steps 6]
"""
from __future__ import annotations

import argparse
import dataclasses
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SETTINGS = [
    ("fixed shape (all off)", dict(enable_bp=0, enable_dp=0, enable_dr=0)),
    ("+ dynamic rerank", dict(enable_bp=0, enable_dp=0, enable_dr=1)),
    ("+ rerank + depth pruning", dict(enable_bp=0, enable_dp=1, enable_dr=1)),
    ("+ rerank + breadth pruning", dict(enable_bp=1, enable_dp=0, enable_dr=1)),
    ("all three", dict(enable_bp=1, enable_dp=1, enable_dr=1)),
]


def run(batches, steps, thresholds):
    import torch
    from paper_2510_26577_b200 import build as _build
    _build.build()
    from paper_2510_26577_b200 import binding, workloads as wl

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    stream = torch.cuda.Stream(device=dev)
    C1, C2, C3 = thresholds
    print("| B | setting | n_i per layer | layers | N | tree build µs | attention µs/layer | attention µs per verified token |")
    print("|---|---|---|---|---|---|---|---|")
    for B in batches:
        w = dataclasses.replace(wl.CONFIGS[f"c3_llama8b_b{B}"], n_layers=2)
        H, K, Ncap = w.depth, w.top_k, w.max_tree
        root, kv0 = wl.root_tokens(w, dev), wl.kv_lengths(w, dev)
        kv_len = kv0.clone()
        q = wl.query(w, 0, dev)
        kvs = [wl.kv_cache(w, l, dev) for l in range(w.n_layers)]
        table, num_pages = wl.page_table(w, dev)
        seq_cap = wl.seq_capacity(w) // w.page_size
        out = torch.zeros_like(q)
        for name, flags in SETTINGS:
            ctx = binding.CastContext(max_batch=B, vocab=w.vocab, top_k=K, max_depth=H, total_token=w.total_token,
                                      max_tree=Ncap, C1=C1, C2=C2, C3=C3, **flags)
            ctx.cast_set_cost_tables(B, *wl.cost_table_arrays(w, B))
            ctx.cast_reserve_attention(q.dtype, B, w.q_heads, w.kv_heads, w.head_dim, w.page_size, seq_cap)
            nt = torch.empty((B, K), dtype=torch.int32, device=dev)
            npr = torch.empty_like(nt)
            cnt = torch.empty((1,), dtype=torch.int32, device=dev)
            tr = [torch.empty((B, Ncap), dtype=torch.int32, device=dev) for _ in range(4)]
            anc = torch.empty((B, Ncap, ctx.words), dtype=torch.int32, device=dev)
            n_tree = torch.empty((B,), dtype=torch.int32, device=dev)

            def tree_build(logits):
                ctx.cast_step_begin(B, root, kv_len)
                for i in range(H):
                    ctx.cast_tree_expand(i + 1, logits[i], nt, npr, cnt)
                ctx.cast_select_nodes(tr[0], tr[1], tr[2], anc, tr[3], None, n_tree)

            def attention():
                for k, v in kvs:
                    ctx.cast_tree_attention(q, k, v, B, w.q_heads, w.kv_heads, w.head_dim, w.page_size, table, seq_cap,
                                            num_pages, kv_len, anc, n_tree, 0.0, out)

            with torch.cuda.stream(stream):
                # a few steps on fresh logits fill the depth-pruning buffers (they persist across steps)
                for s in range(steps):
                    logits = [wl.draft_logits(w, 10 * s + l, dev, peaked=True) for l in range(1, H + 1)]
                    tree_build(logits)
                attention()
                stream.synchronize()
                st, detail = ctx.cast_poll_status()
                assert st == 0, (st, detail)
                info = ctx.cast_step_info()
                N = int(n_tree[0].item())
                gt, ga = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
                with torch.cuda.graph(gt, stream=stream):
                    tree_build(logits)
                with torch.cuda.graph(ga, stream=stream):
                    attention()
                times = []
                for g, reps in ((gt, 50), (ga, 20)):
                    for _ in range(3):
                        g.replay()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    for _ in range(reps):
                        g.replay()
                    e1.record(stream)
                    stream.synchronize()
                    times.append(e0.elapsed_time(e1) * 1e3 / reps)
            us_tree, us_attn = times[0], times[1] / w.n_layers
            n_hist = info["n_hist"][:info["layers"]]
            print(f"| {B} | {name} | {' '.join(str(x) for x in n_hist)} | {info['layers']} | {N} | {us_tree:.0f} | "
                  f"{us_attn:.1f} | {us_attn / (B * N):.3f} |", flush=True)
            ctx.close()
            del gt, ga


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batches", default="1,4,16,64")
    ap.add_argument("--steps", type=int, default=6)
    ap.add_argument("--thresholds", default="1,1,1", help="C1,C2,C3")
    args = ap.parse_args()
    run([int(x) for x in args.batches.split(",")], args.steps, [float(x) for x in args.thresholds.split(",")])


if __name__ == "__main__":
    main()
