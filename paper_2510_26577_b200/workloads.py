"""Seeded synthetic inputs for the CAST draft-and-verify step.

This module only draws random tensors with the shapes, dtypes and value
distributions of Llama/Qwen-style serving workloads and describes the five
benchmark configurations.  It contains none of the method's arithmetic and
imports neither the CUDA binding nor the CPU oracle; both sides of a parity
test receive the very same tensors from here.

The paper evaluates trained draft/target models on public datasets; the hot
path only ever sees logits, Q, K, V tensors and a cost table, so seeded
Gaussian tensors of the right shapes stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

BASE_SEED = 2510_26577 * 10

_TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    batch: int
    kv_dtype: str  # dtype of Q, K, V and the attention output: "f32" | "bf16"
    logit_dtype: str  # dtype of draft and target logits
    q_heads: int
    kv_heads: int
    head_dim: int
    kv_len_lo: int  # prefix lengths are integers uniform in [lo, hi]
    kv_len_hi: int
    page_size: int  # 0 = contiguous cache [B, Lmax, Hkv, D]
    vocab: int
    logit_std: float
    depth: int  # H
    top_k: int  # K
    total_token: int  # m (root included)
    cost_model: bool  # breadth pruning + dynamic rerank driven by the synthetic cost table
    n_layers: int  # verification layers timed per step (distinct KV buffers)
    max_tree: int = 128
    tau: float = 1.4e-4  # slope of the synthetic cost table in B*n
    seed_salt: int = 0  # the first salt whose seed keeps every tree decision of the ORACLE clear of its threshold
    # (tests/seed_margin_audit.py prints the margins of the salts passed over)

    @property
    def seed(self) -> int:
        return BASE_SEED + self.config_id + 1000 * self.seed_salt

    @property
    def gqa(self) -> int:
        return self.q_heads // self.kv_heads


def _c3(batch: int, sub: int, salt: int = 0) -> Workload:
    return Workload(f"c3_llama8b_b{batch}", 30 + sub, batch, "bf16", "f32", 32, 8, 128, 512, 4096, 16,
                    128256, 3.0, 6, 8, 64, True, max(2, 64 // batch), seed_salt=salt)


def _c4(m: int, sub: int) -> Workload:
    return Workload(f"c4_llama70b_n{m}", 40 + sub, 8, "bf16", "f32", 64, 8, 128, 4096, 4096, 0,
                    32000, 3.0, 7, 8, m, False, 4)


CONFIGS: Dict[str, Workload] = {
    w.name: w
    for w in [
        Workload("c1_tiny", 1, 1, "f32", "f32", 8, 8, 64, 256, 256, 0, 4096, 2.0, 4, 4, 16, False, 2),
        Workload("c2_llama8b", 2, 1, "bf16", "f32", 32, 8, 128, 2048, 2048, 0, 128256, 3.0, 6, 10, 60, False, 32),
        _c3(1, 0, 2), _c3(4, 1), _c3(16, 2), _c3(64, 3, 4),
        _c4(16, 0), _c4(32, 1), _c4(64, 2), _c4(128, 3),
        Workload("c5_qwen_long", 5, 4, "bf16", "f32", 28, 4, 128, 32768, 32768, 16, 152064, 3.0, 8, 8, 96, False, 2,
                 seed_salt=1),
    ]
}


def shrink(w: Workload, **kw) -> Workload:
    """A smaller variant of a configuration (for CPU-seconds parity cases)."""
    return replace(w, **kw)


def _gen(w: Workload, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(w.seed * 1000 + stream)
    return g


def _randn(shape, std, dtype, gen, device) -> torch.Tensor:
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if std != 1.0:
        x = x * std
    return x.to(_TORCH_DTYPE[dtype])


def root_tokens(w: Workload, device="cpu") -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed * 1000 + 1)
    return torch.randint(0, w.vocab, (w.batch,), generator=g, dtype=torch.int32).to(device)


def kv_lengths(w: Workload, device="cpu") -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed * 1000 + 2)
    return torch.randint(w.kv_len_lo, w.kv_len_hi + 1, (w.batch,), generator=g, dtype=torch.int32).to(device)


def draft_logits(w: Workload, layer: int, device="cpu", peaked: bool = False, width: int = 0) -> torch.Tensor:
    """[B, W, V] draft logits of one layer (W = `width`, default K rows).  With
    `peaked`, one token per row is raised by 8 so that scores decay slowly with
    depth, as those of a trained draft head do."""
    g = _gen(w, 100 + layer, device)
    rows = width or w.top_k
    x = _randn((w.batch, rows, w.vocab), w.logit_std, "f32", g, device)
    if peaked:
        idx = torch.randint(0, w.vocab, (w.batch, rows, 1), generator=g, device=device)
        x.scatter_add_(2, idx, torch.full_like(idx, 8.0, dtype=torch.float32))
    return x.to(_TORCH_DTYPE[w.logit_dtype])


def query(w: Workload, layer: int, device="cpu") -> torch.Tensor:
    return _randn((w.batch, w.max_tree, w.q_heads, w.head_dim), 1.0, w.kv_dtype, _gen(w, 300 + layer, device), device)


def seq_capacity(w: Workload) -> int:
    """Positions reserved per sequence: the longest prefix plus the tree."""
    cap = w.kv_len_hi + w.max_tree
    if w.page_size:
        cap = (cap + w.page_size - 1) // w.page_size * w.page_size
    return cap


def page_table(w: Workload, device="cpu") -> Tuple[Optional[torch.Tensor], int]:
    """(page_table [B, max_pages] int32, num_pages).  Pages are handed out in a
    seeded random permutation of the pool, so sequences are not contiguous."""
    if w.page_size == 0:
        return None, 0
    per_seq = seq_capacity(w) // w.page_size
    num_pages = per_seq * w.batch
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed * 1000 + 3)
    perm = torch.randperm(num_pages, generator=g, dtype=torch.int64).to(torch.int32)
    return perm.view(w.batch, per_seq).contiguous().to(device), num_pages


def kv_cache(w: Workload, layer: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """K and V ~ N(0,1) for one layer; the tree tokens' rows are part of it
    (positions L_b .. L_b+N-1 are 'already written')."""
    if w.page_size:
        shape = (seq_capacity(w) // w.page_size * w.batch, w.page_size, w.kv_heads, w.head_dim)
    else:
        shape = (w.batch, seq_capacity(w), w.kv_heads, w.head_dim)
    g = _gen(w, 500 + layer, device)
    return _randn(shape, 1.0, w.kv_dtype, g, device), _randn(shape, 1.0, w.kv_dtype, g, device)


def target_logits(w: Workload, device="cpu") -> torch.Tensor:
    return _randn((w.batch, w.max_tree, w.vocab), w.logit_std, w.logit_dtype, _gen(w, 700, device), device)


def plant_acceptance(w: Workload, logits: torch.Tensor, tokens, parent, n_tree, p_plant=0.7, p_geo=0.6) -> None:
    """Make a random tree accept non-trivially: for every tree node that has
    children, with probability p_plant raise the target logit of one child's
    token (child rank geometric with parameter p_geo) to (row max + 1).  The
    tree (tokens, parent, n_tree: host arrays) is an input of this recipe."""
    rng = np.random.Generator(np.random.Philox(w.seed * 1000 + 900))
    tokens = np.asarray(tokens)
    parent = np.asarray(parent)
    for b in range(tokens.shape[0]):
        N = int(n_tree[b])
        kids: Dict[int, List[int]] = {}
        for t in range(1, N):
            kids.setdefault(int(parent[b, t]), []).append(t)
        for t in range(N):
            draw = rng.random()
            rank = int(rng.geometric(p_geo)) - 1
            if t not in kids or draw >= p_plant:
                continue
            child = kids[t][min(rank, len(kids[t]) - 1)]
            row = logits[b, t]
            row[int(tokens[b, child])] = (row.float().max() + 1.0).to(row.dtype)


def stochastic_accept_inputs(w: Workload, tokens, parent, n_tree, device="cpu", noise: float = 1.0, n_cap: int = 0):
    """Inputs of the acceptance step at T > 0 for a given tree (host arrays): per-node draft logits
    [B, Ncap, V] whose largest entries at a node are its children's tokens in tree order (children are the
    top of the draft distribution: row maximum + 1, then steps of 0.5 down), target logits = draft logits +
    `noise` * N(0,1) (a draft that approximates its target), and the uniform numbers u_accept [B, Ncap],
    u_bonus [B] (fp64, open interval)."""
    B, Ncap = w.batch, n_cap or w.max_tree
    g = _gen(w, 800, device)
    draft = _randn((B, Ncap, w.vocab), w.logit_std, "f32", g, device)
    tokens = np.asarray(tokens)
    parent = np.asarray(parent)
    for b in range(B):
        kids: Dict[int, List[int]] = {}
        for t in range(1, int(n_tree[b])):
            kids.setdefault(int(parent[b, t]), []).append(t)
        for t, cs in kids.items():
            top = float(draft[b, t].max()) + 1.0
            for j, c in enumerate(cs):
                draft[b, t, int(tokens[b, c])] = top - 0.5 * j
    target = torch.randn(draft.shape, generator=g, device=device, dtype=torch.float32)
    target.mul_(noise).add_(draft)
    rng = np.random.Generator(np.random.Philox(w.seed * 1000 + 801))
    u_accept = rng.uniform(1e-12, 1.0 - 1e-12, size=(B, Ncap))
    u_bonus = rng.uniform(1e-12, 1.0 - 1e-12, size=(B,))
    dt = _TORCH_DTYPE[w.logit_dtype]
    return (target.to(dt), draft.to(dt), torch.from_numpy(u_accept).to(device), torch.from_numpy(u_bonus).to(device))


def cost_table_arrays(w: Workload, B: int, L: int = 512, M: int = 64, Ntab: int = 128,
                      stepped: bool = False, skewed: bool = False) -> Tuple[int, int, int, np.ndarray, np.ndarray]:
    """Synthetic stand-in for the profiled latency tables (the real ones need
    the models): f_T(B, c, n) = 1 + 0.25*B*c/(64*4096) + tau*B*n on the grid
    c = g*L, n = 1..Ntab, and f_D = 0.05 * f_T; strictly increasing in n.  The
    `stepped` variant adds 0.02*ceil(B*n/64) (tile quantisation).

    `skewed` is a test family in which a lookup in the wrong table, the wrong
    grid row or the wrong column changes the numbers visibly: the rows differ
    by tens of percent (so the grid step should be small enough for the
    contexts in play to cross rows), the slope in n grows with the row, and
    f_D is not a multiple of f_T (own offset, convex in n)."""
    c = (np.arange(1, M + 1, dtype=np.float64) * L)[:, None]
    n = np.arange(1, Ntab + 1, dtype=np.float64)[None, :]
    if skewed:
        g = np.arange(1, M + 1, dtype=np.float64)[:, None]
        fT = 1.0 + 0.35 * g + w.tau * B * n * (1.0 + 0.25 * g)
        fD = 0.02 + 0.015 * g * g + 0.4 * w.tau * B * n ** 1.25 / (1.0 + 0.1 * g)
        return L, M, Ntab, fT, fD
    fT = 1.0 + 0.25 * (B * c) / (64.0 * 4096.0) + w.tau * B * n
    if stepped:
        fT = fT + 0.02 * np.ceil(B * n / 64.0)
    fD = 0.05 * fT
    return L, M, Ntab, fT, fD
