"""Shared plumbing of the parity tests: run the same seeded inputs through the
CPU oracle and through the CUDA library (via its C-ABI binding) and compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import CastOracle, CostTable, OracleConfig
from paper_2510_26577_b200 import workloads as wl


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact conversion of an fp32/bf16 tensor to float64 on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def cfg_kwargs(w: wl.Workload, **over):
    kw = dict(vocab=w.vocab, top_k=w.top_k, max_depth=w.depth, total_token=w.total_token, max_tree=w.max_tree)
    if w.cost_model:
        kw.update(enable_bp=1, enable_dr=1)
    kw.update(over)
    return kw


def make_tables(w: wl.Workload, B: int, stepped=False, skewed=False):
    if skewed:  # a fine grid, so that the tree's own context (tens of nodes) and the ragged prefixes cross rows
        return wl.cost_table_arrays(w, B, L=8, M=48, Ntab=64, skewed=True)
    L, M, Ntab, fT, fD = wl.cost_table_arrays(w, B, stepped=stepped)
    return L, M, Ntab, fT, fD


# ------------------------------------------------------------------ tree build
def oracle_tree(kw, tables, root, kv_len, logits_layers, oracle=None):
    """logits_layers: list of [B, W, V] tensors (any dtype).  Returns dict."""
    o = oracle or CastOracle(OracleConfig(**kw), tables)
    o.step_begin(root.cpu().numpy(), kv_len.cpu().numpy())
    per_layer = []
    for i, lg in enumerate(logits_layers, start=1):
        nt, npr, cnt = o.expand(i, to_f64(lg))
        per_layer.append((nt, npr, cnt))
    sel = o.select_nodes()
    sel["per_layer"] = per_layer
    sel["n_hist"] = list(o.n_hist[1:])
    sel["pool_size"] = o.pool_size
    sel["min_score_gap"] = o.min_score_gap
    sel["stable"] = o.stable
    sel["oracle"] = o
    return sel


def alloc_tree_outputs(B, Ncap, words, device="cuda"):
    return dict(
        tokens=torch.empty((B, Ncap), dtype=torch.int32, device=device),
        parent=torch.empty((B, Ncap), dtype=torch.int32, device=device),
        depth=torch.empty((B, Ncap), dtype=torch.int32, device=device),
        anc=torch.empty((B, Ncap, words), dtype=torch.int32, device=device),
        pool_idx=torch.empty((B, Ncap), dtype=torch.int32, device=device),
        scores=torch.empty((B, Ncap), dtype=torch.float64, device=device),
        n_tree=torch.empty((B,), dtype=torch.int32, device=device),
    )


def gpu_tree(ctx, root, kv_len, logits_layers):
    B = root.shape[0]
    W = ctx.width
    per_layer = []
    ctx.cast_step_begin(B, root, kv_len)
    for i, lg in enumerate(logits_layers, start=1):
        nt = torch.empty((B, W), dtype=torch.int32, device="cuda")
        npr = torch.empty((B, W), dtype=torch.int32, device="cuda")
        cnt = torch.empty((1,), dtype=torch.int32, device="cuda")
        ctx.cast_tree_expand(i, lg, nt, npr, cnt)
        per_layer.append((nt, npr, cnt))
    out = alloc_tree_outputs(B, ctx.cfg.max_tree, ctx.words)
    ctx.cast_select_nodes(out["tokens"], out["parent"], out["depth"], out["anc"], out["pool_idx"], out["scores"],
                          out["n_tree"])
    status = ctx.cast_poll_status()
    info = ctx.cast_step_info()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    res["anc"] = res["anc"].view(np.uint32)
    res["per_layer"] = [(a.cpu().numpy(), b.cpu().numpy(), int(c.item())) for a, b, c in per_layer]
    res["status"] = status
    res["info"] = info
    res["dev"] = out
    return res


def assert_tree_equal(g, o, score_tol=5e-6):
    """Bit-exact structure; log-values within score_tol."""
    assert g["status"][0] == 0, f"device status {g['status']}"
    L = len(o["n_hist"])
    assert g["info"]["layers"] == L
    assert g["info"]["n_hist"][:L] == o["n_hist"], (g["info"]["n_hist"], o["n_hist"])
    assert g["info"]["pool_size"] == o["pool_size"]
    for i, ((gt, gp, gc), (ot, op, oc)) in enumerate(zip(g["per_layer"], o["per_layer"])):
        assert gc == oc, f"layer {i + 1}: next_count {gc} vs {oc}"
        if i < L:
            assert np.array_equal(gt, ot), f"layer {i + 1}: next_tokens"
            assert np.array_equal(gp, op), f"layer {i + 1}: next_parent_row"
    assert np.array_equal(g["n_tree"], o["n_tree"]), (g["n_tree"], o["n_tree"])
    for k in ("tokens", "parent", "depth", "pool_idx", "anc"):
        assert np.array_equal(g[k], o[k]), k
    assert np.max(np.abs(g["scores"] - o["scores"])) < score_tol


# ------------------------------------------------------------------ attention
def gpu_attention(ctx, w, q, k, v, table, num_pages, kv_len, anc, n_tree, scale=0.0, first_row=None):
    out = torch.full_like(q, float("nan"))
    anc_t = anc if torch.is_tensor(anc) else torch.from_numpy(anc.view(np.int32)).cuda()
    ctx.cast_reserve_attention(q.dtype, q.shape[0], w.q_heads, w.kv_heads, w.head_dim, w.page_size,
                               wl.seq_capacity(w) // (w.page_size or 1))
    if first_row is None:
        ctx.cast_tree_attention(q, k, v, q.shape[0], w.q_heads, w.kv_heads, w.head_dim, w.page_size, table,
                                wl.seq_capacity(w) // (w.page_size or 1), num_pages, kv_len, anc_t, n_tree, scale, out)
    else:
        ctx.cast_tree_attention_rows(q, k, v, q.shape[0], w.q_heads, w.kv_heads, w.head_dim, w.page_size, table,
                                     wl.seq_capacity(w) // (w.page_size or 1), num_pages, kv_len, anc_t, n_tree,
                                     first_row, scale, out)
    torch.cuda.synchronize()
    return out


def attention_tolerance(dtype: str) -> float:
    # max-abs error allowed: 1e-5 for fp32 inputs, 2e-2 for bf16 inputs
    return 1e-5 if dtype == "f32" else 2e-2
