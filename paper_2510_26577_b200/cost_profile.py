"""Cost tables S_T(B), S_D(B) measured on the GPU at hand.

The paper profiles f(B, c, n) - the time of one forward over n new tokens per sequence at batch size
B and context length c - for the target and the draft model, on the grid c = L, 2L, ..., ML and
n = 1..N (Sec. "Method"), and notes that this has to be done per model and device.  Without model
trained weights the forward's two dominant parts can still be timed at the model's shapes: this module
times `cast_tree_attention` of this library over the grid, and the dense projections of one decoder
layer (and, for the draft head, the vocabulary projection) as library bf16 GEMMs on random weights of
the workload's dimensions over B * n rows, adds them up per layer and hands the tables to
`cast_set_cost_tables`. Elementwise work (norms, rotary, activation) is left out: it is a few per cent
of a layer and does not change with what the cost model decides between.

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


def measure_layer_gemms_us(w, B: int, n_points=N_POINTS, reps: int = 5, ffn_mult: float = 3.5):
    """(layer_us[j], head_us[j]): microseconds of the dense projections of one decoder layer of the workload's
    dimensions (hidden = q_heads * head_dim; fused QKV, output, gate+up and down projections with an
    intermediate size of ffn_mult * hidden) and of the vocabulary projection, each on B * n_points[j] rows, as
    bf16 library GEMMs on random weights. A layer's weights are several times the L2 cache, so every
    repetition streams them from HBM as a model with many layers does; the vocabulary matrix alone is too."""
    import torch

    dev = torch.device("cuda", torch.cuda.current_device())
    n_points = tuple(n for n in n_points if n <= w.max_tree)
    hidden, kvd = w.q_heads * w.head_dim, w.kv_heads * w.head_dim
    ffn = int(ffn_mult * hidden)
    gen = torch.Generator(device=dev).manual_seed(1234)
    mk = lambda r, c: (torch.randn((r, c), generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)
    w_qkv, w_o, w_gu, w_d, w_lm = mk(hidden, hidden + 2 * kvd), mk(hidden, hidden), mk(hidden, 2 * ffn), mk(ffn, hidden), \
        mk(hidden, w.vocab)

    def layer(x):
        x @ w_qkv
        x @ w_o
        return (x @ w_gu)[:, :ffn] @ w_d

    def timed(fn, x):
        for _ in range(3):
            fn(x)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn(x)
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps

    layer_us, head_us = np.zeros(len(n_points)), np.zeros(len(n_points))
    for j, n in enumerate(n_points):
        x = mk(B * n, hidden)
        layer_us[j] = timed(layer, x)
        head_us[j] = timed(lambda y: y @ w_lm, x)
    return layer_us, head_us


def tables_from_measurement(t: np.ndarray, n_points, B: int, Ntab: int, n_layers: int, gemm_us=(20.0, 0.35),
                            draft_layers: int = 1, layer_us=None, head_us=None) -> Tuple[np.ndarray, np.ndarray]:
    """f_T[g][k] and f_D[g][k], k = 1..Ntab, in microseconds, made strictly increasing in n as Algorithm 1
    requires. A layer = attention interpolated in n + its GEMMs: the measured `layer_us` interpolated likewise,
    or, without a measurement, the linear form a + b*B*n with (a, b) = gemm_us. f_T = n_layers layers;
    f_D = draft_layers layers + the vocabulary projection `head_us` when that was measured (the draft head
    scores the whole vocabulary for every new node, which the target does for accepted tokens only)."""
    M = t.shape[0]
    n = np.arange(1, Ntab + 1, dtype=np.float64)
    pts = np.asarray(n_points, dtype=np.float64)
    attn = np.stack([np.interp(n, pts, t[g]) for g in range(M)])
    gemm = np.interp(n, pts, layer_us) if layer_us is not None else gemm_us[0] + gemm_us[1] * B * n
    layer = attn + gemm[None, :]
    fT, fD = n_layers * layer, draft_layers * layer
    if head_us is not None:
        fD = fD + np.interp(n, pts, head_us)[None, :]
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
    print("| B | f_T(B, L, 1) µs | f_T(B, ML, 1) | f_T(B, ML, 64) | f_D(B, ML, 1) | f_D(B, ML, 64) | layer GEMMs n=1 / 64 | "
          "n_i per layer | N picked (context 2048, peaked logits) |")
    print("|---|---|---|---|---|---|---|---|---|")
    for B in (int(x) for x in args.batches.split(",")):
        w = dataclasses.replace(wl.CONFIGS[f"c3_llama8b_b{B}"], kv_len_lo=2048, kv_len_hi=2048)
        t, pts = measure_attention_us(w, B, L, M)
        layer_us, head_us = measure_layer_gemms_us(w, B, pts)
        Ntab = 128
        fT, fD = tables_from_measurement(t, pts, B, Ntab, n_layers=32, layer_us=layer_us, head_us=head_us)
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
        print(f"| {B} | {fT[0, 0]:.0f} | {fT[M - 1, 0]:.0f} | {fT[M - 1, 63]:.0f} | {fD[M - 1, 0]:.0f} | {fD[M - 1, 63]:.0f} | "
              f"{np.interp(1, pts, layer_us):.0f} / {np.interp(64, pts, layer_us):.0f} | "
              f"{' '.join(str(x) for x in info['n_hist'][:info['layers']])} | {int(n_tree[0].item())} |", flush=True)
        ctx.close()


if __name__ == "__main__":
    main()
