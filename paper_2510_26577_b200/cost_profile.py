"""Cost tables S_T(B), S_D(B) measured on the GPU at hand.

The paper profiles f(B, c, n) - the time of one forward over n new tokens per sequence at batch size
B and context length c - for the target and the draft model, on the grid c = L, 2L, ..., ML and
n = 1..N (Sec. "Method"), and notes that this has to be done per model and device.  Without model
weights the attention part of that forward is the one thing that can be measured for real here:
this module times `cast_tree_attention` of this library over the grid and adds a linear stand-in for
the rest of a layer (the GEMMs: a + b * B * n), then hands the tables to `cast_set_cost_tables`.

  python -m paper_2510_26577_b200.cost_profile [--batches 1,4,16,64]

prints, per batch size, the table's corner values and the tree sizes the cost model then picks.
"""
from __future__ import annotations

import argparse
import dataclasses
import os
import sys
from typing import Tuple

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

N_POINTS = (1, 2, 4, 8, 16, 32, 64, 128)  # tree sizes that are timed; the rest is interpolated


def measure_attention_us(w, B: int, L: int, M: int, n_points=N_POINTS, reps: int = 10, max_bytes: int = 12 << 30):
    """t[g-1][j] = microseconds of one `cast_tree_attention` layer at context g*L and n_points[j] tree
    tokens per sequence (chain trees; the mask's shape does not change the time). Successive calls read
    different KV buffers, enough of them that a buffer has left the L2 cache (more than twice its size has
    been read) before it is used again: the figures are HBM figures, as in a model whose layers each have
    their own cache."""
    import torch
    from paper_2510_26577_b200 import binding, workloads as wl

    dev = torch.device("cuda", torch.cuda.current_device())
    n_points = tuple(n for n in n_points if n <= w.max_tree)
    wb = dataclasses.replace(w, batch=B, kv_len_lo=M * L, kv_len_hi=M * L)
    ctx = binding.CastContext(max_batch=B, vocab=w.vocab, top_k=w.top_k, max_depth=w.depth, total_token=w.max_tree,
                              max_tree=w.max_tree)
    q = wl.query(wb, 0, dev)
    k0, v0 = wl.kv_cache(wb, 0, dev)
    table, num_pages = wl.page_table(wb, dev)
    seq_cap = wl.seq_capacity(wb) // (wb.page_size or 1)
    ctx.cast_reserve_attention(q.dtype, B, w.q_heads, w.kv_heads, w.head_dim, w.page_size, seq_cap)
    l2 = int(torch.cuda.get_device_properties(dev).L2_cache_size)
    row_bytes = 2 * w.kv_heads * w.head_dim * k0.element_size()  # K and V of one position

    def buffers_needed(ctx_len):
        return -(-2 * l2 // max(B * ctx_len * row_bytes, 1)) + 1

    buf_bytes = 2 * k0.numel() * k0.element_size()
    nbuf = max(2, min(buffers_needed(L), 128, max_bytes // buf_bytes))
    ks = [k0] + [torch.randn_like(k0) for _ in range(nbuf - 1)]
    vs = [v0] + [torch.randn_like(v0) for _ in range(nbuf - 1)]
    out = torch.empty_like(q)
    words = ctx.words
    stream = torch.cuda.Stream(device=dev)
    t = np.zeros((M, len(n_points)))
    with torch.cuda.stream(stream):
        for j, n in enumerate(n_points):
            anc = np.zeros((B, w.max_tree, words), dtype=np.uint32)
            for i in range(n):  # chain: token i sees tokens 0..i
                for a in range(i + 1):
                    anc[:, i, a >> 5] |= np.uint32(1 << (a & 31))
            anc_t = torch.from_numpy(anc.view(np.int32)).to(dev)
            n_tree = torch.full((B,), n, dtype=torch.int32, device=dev)
            for g in range(1, M + 1):
                kv_len = torch.full((B,), g * L, dtype=torch.int32, device=dev)
                use = max(2, min(nbuf, buffers_needed(g * L)))
                call = lambda i: ctx.cast_tree_attention(q, ks[i % use], vs[i % use], B, w.q_heads, w.kv_heads, w.head_dim,
                                                         w.page_size, table, seq_cap, num_pages, kv_len, anc_t, n_tree,
                                                         0.0, out)
                for i in range(3):
                    call(i)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for i in range(reps):
                    call(3 + i)
                e1.record(stream)
                stream.synchronize()
                t[g - 1, j] = e0.elapsed_time(e1) * 1e3 / reps
        assert ctx.cast_poll_status()[0] == 0
    ctx.close()
    return t, n_points


def tables_from_measurement(t: np.ndarray, n_points, B: int, Ntab: int, n_layers: int, gemm_us=(20.0, 0.35),
                            draft_layers: int = 1) -> Tuple[np.ndarray, np.ndarray]:
    """f_T[g][k] and f_D[g][k], k = 1..Ntab: n_layers x (attention interpolated in n + the linear GEMM
    stand-in a + b*B*n microseconds), made strictly increasing in n as Algorithm 1 requires."""
    M = t.shape[0]
    n = np.arange(1, Ntab + 1, dtype=np.float64)
    attn = np.stack([np.interp(n, np.asarray(n_points, dtype=np.float64), t[g]) for g in range(M)])
    layer = attn + gemm_us[0] + gemm_us[1] * B * n[None, :]
    fT, fD = n_layers * layer, draft_layers * layer
    for f in (fT, fD):
        for k in range(1, Ntab):
            f[:, k] = np.maximum(f[:, k], f[:, k - 1] * (1.0 + 1e-6))
    return fT, fD


def main():
    import torch
    from paper_2510_26577_b200 import build as _build
    _build.build()
    from paper_2510_26577_b200 import binding, workloads as wl

    ap = argparse.ArgumentParser()
    ap.add_argument("--batches", default="1,4,16,64")
    ap.add_argument("--grid", default="512,8", help="L,M: contexts L, 2L, ..., ML")
    ap.add_argument("--threshold", type=float, default=0.1, help="C1 = C2 = C3")
    args = ap.parse_args()
    L, M = (int(x) for x in args.grid.split(","))
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    print("| B | f_T(B, L, 1) µs | f_T(B, ML, 1) | f_T(B, ML, 64) | n_i per layer | N picked (context 2048, peaked logits) |")
    print("|---|---|---|---|---|---|")
    for B in (int(x) for x in args.batches.split(",")):
        w = dataclasses.replace(wl.CONFIGS[f"c3_llama8b_b{B}"], kv_len_lo=2048, kv_len_hi=2048)
        t, pts = measure_attention_us(w, B, L, M)
        Ntab = 128
        fT, fD = tables_from_measurement(t, pts, B, Ntab, n_layers=32)
        ctx = binding.CastContext(max_batch=B, vocab=w.vocab, top_k=w.top_k, max_depth=w.depth,
                                  total_token=w.total_token, C1=args.threshold, C2=args.threshold, C3=args.threshold,
                                  enable_bp=1, enable_dr=1)
        ctx.cast_set_cost_tables(B, L, M, Ntab, fT, fD)
        root, kv = wl.root_tokens(w, dev), wl.kv_lengths(w, dev)
        K, H, Ncap = w.top_k, w.depth, w.max_tree
        nt = torch.empty((B, K), dtype=torch.int32, device=dev)
        npr, cnt = torch.empty_like(nt), torch.empty((1,), dtype=torch.int32, device=dev)
        tr = [torch.empty((B, Ncap), dtype=torch.int32, device=dev) for _ in range(4)]
        anc = torch.empty((B, Ncap, ctx.words), dtype=torch.int32, device=dev)
        n_tree = torch.empty((B,), dtype=torch.int32, device=dev)
        ctx.cast_step_begin(B, root, kv)
        for i in range(H):
            ctx.cast_tree_expand(i + 1, wl.draft_logits(w, i + 1, dev, peaked=True), nt, npr, cnt)
        ctx.cast_select_nodes(tr[0], tr[1], tr[2], anc, tr[3], None, n_tree)
        torch.cuda.synchronize()
        assert ctx.cast_poll_status()[0] == 0
        info = ctx.cast_step_info()
        print(f"| {B} | {fT[0, 0]:.0f} | {fT[M - 1, 0]:.0f} | {fT[M - 1, 63]:.0f} | "
              f"{' '.join(str(x) for x in info['n_hist'][:info['layers']])} | {int(n_tree[0].item())} |", flush=True)
        ctx.close()


if __name__ == "__main__":
    main()
