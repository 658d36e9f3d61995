"""Plain float64 CPU oracle of one CAST draft-and-verify step (numpy only).

TEST INFRASTRUCTURE.  Not part of the product path; shares no code with the
CUDA library.  Every function follows either the paper's algorithm in the
paper's order and notation (tree sizing: Eq. 1, Eq. 2, Algorithm 1, the depth
pruning rule, the dynamic rerank) or the plain definition of the quantity where
the paper only names it (top-K children, softmax attention under the ancestor
mask, greedy acceptance, a KV gather).

Notation (paper, Section "Method"): B batch rows, K children per node, H draft
layers, N_i candidates of layer i, n_i retained nodes of layer i, m cap on the
verified tokens, v(u) node value, u_k utility, c_k normalised cost.

Pins (tests marked "not gpu"): Algorithm 1 on hand-worked cases and on the
Theorem's linear-cost special case in exact rational arithmetic; select() on a
hand table; expansion and rerank against brute-force enumeration of all paths
on tiny vocabularies; the composition of Eq. 1, Eq. 2, Algorithm 1, the depth
test and the rerank inside expand() / select_nodes() with every sizing switch
on against a batch-2, two-step case worked by hand in exact fractions (ragged
prefixes, cost rows that all differ, f_D not proportional to f_T, C1 != C3),
and the orders of exactly equal values and the ">=" of the depth test against
hand-worked exact-tie cases (tests/golden/cast_step_*.txt); attention against separately coded causal attention on a
chain tree and against per-path dense attention; acceptance against sequential
token-by-token decoding; stochastic acceptance against a hand-worked case, the
greedy rule for a one-hot target, the all-accept case P_T = P_D and the
output-distribution-equals-P_T property on sampled trees; compaction against an
out-of-place gather.
Parity unpinned: the FIFO length R, the split of the paper's single reported
"threshold" into C1, C2, C3, and the cost-table contents - the paper prints no
value for any of them, so they are parameters here, not results.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np


# --------------------------------------------------------------------------
# Cost model (Section "Method": f(B,c,n), select(c), tables S_T(B), S_D(B))
# --------------------------------------------------------------------------
def select_grid(c: int, L: int, M: int) -> int:
    """Grid row g in [1, M] such that select(c) = g * L.

    The paper prints select(c) = (max(floor(c/L), M-1) + 1) L; with `max` every
    lookup would land on or beyond the last of the M table rows, so the operator
    is read as `min`: round c up to the next multiple of L and clamp to M*L.
    """
    return min(c // L, M - 1) + 1


@dataclass
class CostTable:
    """S_T(B) and S_D(B) for one batch size B: f(B, g*L, n), g=1..M, n=1..Ntab."""

    B: int
    L: int
    M: int
    Ntab: int
    fT: np.ndarray  # [M, Ntab] float64, target-model cost
    fD: np.ndarray  # [M, Ntab] float64, draft-model cost

    def __post_init__(self):
        self.fT = np.asarray(self.fT, dtype=np.float64).reshape(self.M, self.Ntab)
        self.fD = np.asarray(self.fD, dtype=np.float64).reshape(self.M, self.Ntab)
        # Algorithm 1 requires c strictly increasing in n.
        for name, f in (("fT", self.fT), ("fD", self.fD)):
            if not np.all(np.isfinite(f)) or np.any(f <= 0):
                raise ValueError(f"{name} must be finite and positive")
            if self.Ntab > 1 and np.any(np.diff(f, axis=1) <= 0):
                raise ValueError(f"{name} must be strictly increasing in n")


def alg1_select_max_valid_index(u, c, C: float, slack: float = 0.0) -> int:
    """Algorithm 1 ("Select Maximum Valid Index").  u, c hold u[1..n], c[1..n]
    (python index k-1 holds element k), c strictly increasing.

    What the algorithm computes: index j is valid iff every chord from an
    earlier index i < j has slope (u[j]-u[i])/(c[j]-c[i]) >= C (a cleared index
    still clears later ones; index 1 has no earlier index and is always valid);
    the result is the largest valid index.  The slope test is written
    division-free (the denominator is positive) and strict: a slope of exactly
    C keeps the index.  `slack` shifts every test by slack*(|u[j]|+|u[i]|); it
    is 0 for the algorithm proper and is used only by alg1_is_stable.
    """
    n = len(u)
    assert n >= 1 and len(c) == n

    def chord_ok(i, j):
        bound = C * (c[j] - c[i])
        if slack != 0.0:
            bound = bound + slack * (abs(u[j]) + abs(u[i]))
        return not (u[j] - u[i] < bound)

    valid = [j for j in range(n) if all(chord_ok(i, j) for i in range(j))]
    return valid[-1] + 1


def alg1_is_stable(u, c, C: float, rel: float = 2e-6) -> bool:
    """True when no perturbation of the utilities of relative size `rel` can
    change Algorithm 1's output (the marks are monotone in the slack)."""
    return alg1_select_max_valid_index(u, c, C, +rel) == alg1_select_max_valid_index(u, c, C, -rel)


# --------------------------------------------------------------------------
# Draft distribution pieces (Section "Tree Expansion Phase")
# --------------------------------------------------------------------------
def log_sum_exp(x: np.ndarray) -> float:
    """log sum_t exp(x_t): the normaliser of P_D over the full vocabulary."""
    m = np.max(x)
    return float(m + np.log(np.sum(np.exp(x - m))))


def topk_children(x: np.ndarray, K: int) -> np.ndarray:
    """The K tokens first in the order (logit descending, token id ascending)."""
    order = np.argsort(-x, kind="stable")  # full stable sort of the V pairs
    return order[:K]


def ancestor_masks(parent: np.ndarray, N: int, words: int) -> np.ndarray:
    """anc[t] = bit set of t and all of its ancestors (parent[root] = -1)."""
    anc = np.zeros((len(parent), words), dtype=np.uint32)
    for t in range(N):
        a = t
        while a >= 0:
            anc[t, a // 32] |= np.uint32(1 << (a % 32))
            a = int(parent[a])
    return anc


@dataclass
class OracleConfig:
    vocab: int
    top_k: int  # K
    max_depth: int  # H
    total_token: int  # m
    max_width: int = 0  # W (0 -> K)
    max_tree: int = 128  # Ncap
    C1: float = 1.0
    C2: float = 1.0
    C3: float = 1.0
    fifo_len: int = 8  # R
    enable_bp: int = 0
    enable_dp: int = 0
    enable_dr: int = 0
    pool_mode: int = 0  # 0: every generated candidate + root; 1: root + retained nodes only
    ctx_base_mode: int = 0  # 0: Eq. 2 context = sum_{j<i} n_j; 1: add n_0
    rerank_per_row: int = 0  # 1: every sequence runs the rerank on its own values (N differs per sequence)

    @property
    def width(self) -> int:
        return self.max_width if self.max_width > 0 else self.top_k


class CastOracle:
    """Tree construction state machine: step_begin, expand (once per layer),
    select_nodes.  Cross-step state: the depth-pruning FIFO buffers A_i."""

    def __init__(self, cfg: OracleConfig, tables: Optional[Dict[int, CostTable]] = None):
        self.cfg = cfg
        self.tables = tables or {}
        # A_i for i = 1..H-1, each initialised with {1}.
        self.fifo: List[List[float]] = [[1.0] for _ in range(max(cfg.max_depth - 1, 0))]
        self.B = 0

    # -- helpers ------------------------------------------------------------
    def _table(self) -> CostTable:
        if self.B not in self.tables:
            raise KeyError(f"no cost table for batch size {self.B}")
        return self.tables[self.B]

    # -- step ---------------------------------------------------------------
    def step_begin(self, root_token, kv_len):
        root_token = np.asarray(root_token)
        kv_len = np.asarray(kv_len)
        self.B = int(root_token.shape[0])
        cfg = self.cfg
        if cfg.enable_bp or cfg.enable_dp or cfg.enable_dr:
            self._table()
        # pool per row: root has value 1 (log 0), depth 0.
        self.score = [[0.0] for _ in range(self.B)]
        self.token = [[int(root_token[b])] for b in range(self.B)]
        self.parent = [[-1] for _ in range(self.B)]
        self.depth = [[0] for _ in range(self.B)]
        self.kept_flag = [[True] for _ in range(self.B)]
        self.retained = [[0] for _ in range(self.B)]  # pool indices, rank order
        self.pool_size = 1
        self.n_prev = 1
        self.n_hist = [1]  # n_0 counts the root as one node of layer 0
        self.ctx_sum = 0  # sum_{j=1}^{i-1} n_j
        self.n0 = int(np.max(kv_len)) if self.B else 0  # padded context length
        self.u_last = 1.0
        self.layers_done = 0
        # decision margins of this step (test bookkeeping, not part of the method)
        self.min_score_gap = float("inf")
        self.stable = True

    def _note_gaps(self, sorted_scores: np.ndarray, upto: int):
        for k in range(min(upto, len(sorted_scores) - 1)):
            g = sorted_scores[k] - sorted_scores[k + 1]
            if g > 0.0:
                self.min_score_gap = min(self.min_score_gap, float(g))

    def expand(self, layer: int, logits: np.ndarray):
        """One layer of the expansion stage.  logits: [B, W, V] float64; row r of
        batch row b belongs to the rank-r retained node of the previous layer."""
        cfg = self.cfg
        B, K, W, H = self.B, cfg.top_k, cfg.width, cfg.max_depth
        next_tokens = np.full((B, W), -1, dtype=np.int32)
        next_parent_row = np.full((B, W), -1, dtype=np.int32)
        if self.n_prev == 0 or layer > H:
            return next_tokens, next_parent_row, 0
        assert layer == self.layers_done + 1
        n_prev = self.n_prev
        base = self.pool_size
        # children: top-K of P_D(.|c_u); value = product along the path (log domain)
        for b in range(B):
            for r in range(n_prev):
                p = self.retained[b][r]
                x = np.asarray(logits[b, r], dtype=np.float64)
                if np.any(np.isnan(x)) or np.any(x == np.inf):
                    raise FloatingPointError("non-finite draft logit")
                lse = log_sum_exp(x)
                for tok in topk_children(x, K):
                    self.score[b].append(self.score[b][p] + (float(x[tok]) - lse))
                    self.token[b].append(int(tok))
                    self.parent[b].append(p)
                    self.depth[b].append(layer)
                    self.kept_flag[b].append(False)
        N_i = n_prev * K
        # per-row descending sort of the N_i candidates
        order = []
        for b in range(B):
            cand = list(range(base, base + N_i))
            cand.sort(key=lambda p: (-self.score[b][p], self.token[b][p], p))
            order.append(cand)
        need_cost = bool(cfg.enable_bp or cfg.enable_dp)
        n = min(N_i, W)
        if need_cost:
            n = min(n, self._table().Ntab)
        # Eq. 1: u_k = (1/B) sum_j sum_{s<=k} v_i^(j)(s)
        v = np.array([[np.exp(self.score[b][order[b][s]]) for s in range(n)] for b in range(B)])
        u = np.cumsum(v, axis=1).sum(axis=0) / B
        for b in range(B):
            self._note_gaps(np.array([self.score[b][p] for p in order[b]]), n)
        # Eq. 2: c_k = S_D(B)[select(ctx)][k] / S_T(B)[select(ctx)][1]
        c = None
        if need_cost:
            tab = self._table()
            ctx = self.ctx_sum + (self.n0 if cfg.ctx_base_mode else 0)
            g = select_grid(ctx, tab.L, tab.M)
            c = tab.fD[g - 1, :n] / tab.fT[g - 1, 0]
        # breadth pruning
        if cfg.enable_bp:
            n_i = alg1_select_max_valid_index(u, c, cfg.C1)
            self.stable &= alg1_is_stable(u, c, cfg.C1)
        else:
            n_i = n
        # depth pruning: gain ratio of the layer just sized goes into A_{i-1};
        # alpha_i is read from A_i, which this call does not touch.
        go = True
        if cfg.enable_dp:
            if layer >= 2:
                phi = u[n_i - 1] / self.u_last
                A = self.fifo[layer - 2]
                A.append(float(phi))
                if len(A) > cfg.fifo_len:
                    A.pop(0)
            if layer < H:
                alpha = float(np.mean(self.fifo[layer - 1]))
                lhs = alpha * u[n_i - 1] / c[n_i - 1]
                go = bool(lhs >= cfg.C2)
                if abs(lhs - cfg.C2) < 2e-6 * max(abs(lhs), abs(cfg.C2)):
                    self.stable = False
        for b in range(B):
            self.retained[b] = order[b][:n_i]
            for s, p in enumerate(self.retained[b]):
                self.kept_flag[b][p] = True
                next_tokens[b, s] = self.token[b][p]
                next_parent_row[b, s] = (p - base) // K
        next_count = n_i if (layer < H and go) else 0
        self.n_hist.append(n_i)
        self.n_prev = next_count
        self.ctx_sum += n_i
        self.u_last = float(u[n_i - 1])
        self.pool_size += N_i
        self.layers_done = layer
        self.last_u, self.last_c = u, c
        return next_tokens, next_parent_row, next_count

    def select_nodes(self):
        """Dynamic rerank + linearisation.  Returns a dict of [B, Ncap] arrays."""
        cfg = self.cfg
        B, Ncap = self.B, cfg.max_tree
        words = (Ncap + 31) // 32
        order = []
        for b in range(B):
            if cfg.pool_mode == 0:
                members = list(range(self.pool_size))
            else:
                members = [p for p in range(self.pool_size) if self.kept_flag[b][p]]
            members.sort(key=lambda p: (-self.score[b][p], self.depth[b][p], self.token[b][p], p))
            order.append(members)
        P = len(order[0]) if B else 0
        n = min(P, cfg.total_token, Ncap)
        if cfg.enable_dr:
            n = min(n, self._table().Ntab)
        vb = np.array([[np.exp(self.score[b][order[b][s]]) for s in range(n)] for b in range(B)])
        u_mean = np.cumsum(vb.mean(axis=0))  # Eq. 1: batch mean of the rank-wise values
        for b in range(B):
            self._note_gaps(np.array([self.score[b][p] for p in order[b]]), n)
        if cfg.enable_dr:
            tab = self._table()
            g0 = select_grid(self.n0, tab.L, tab.M)
            c = tab.fT[g0 - 1, :n] / tab.fT[g0 - 1, 0]
            if cfg.rerank_per_row:  # u from the sequence's own values instead of the batch mean of Eq. 1
                Nb = []
                for b in range(B):
                    u = np.cumsum(vb[b])
                    Nb.append(alg1_select_max_valid_index(u, c, cfg.C3))
                    self.stable &= alg1_is_stable(u, c, cfg.C3)
            else:
                Nb = [alg1_select_max_valid_index(u_mean, c, cfg.C3)] * B
                self.stable &= alg1_is_stable(u_mean, c, cfg.C3)
        else:
            Nb = [n] * B
        out = {
            "tokens": np.full((B, Ncap), -1, dtype=np.int32),
            "parent": np.full((B, Ncap), -1, dtype=np.int32),
            "depth": np.full((B, Ncap), -1, dtype=np.int32),
            "anc": np.zeros((B, Ncap, words), dtype=np.uint32),
            "pool_idx": np.full((B, Ncap), -1, dtype=np.int32),
            "scores": np.zeros((B, Ncap), dtype=np.float64),
            "n_tree": np.array(Nb, dtype=np.int32),
        }
        for b in range(B):
            N = Nb[b]
            kept = sorted(order[b][:N])  # ascending pool index: root first, parents before children
            lin = {p: t for t, p in enumerate(kept)}
            for t, p in enumerate(kept):
                out["tokens"][b, t] = self.token[b][p]
                pp = self.parent[b][p]
                if pp >= 0:
                    assert pp in lin, "kept node whose parent was dropped"
                    out["parent"][b, t] = lin[pp]
                out["depth"][b, t] = self.depth[b][p]
                out["pool_idx"][b, t] = p
                out["scores"][b, t] = self.score[b][p]
            out["anc"][b] = ancestor_masks(out["parent"][b], N, words)
        self.last_u_sel = u_mean
        self.last_c_sel = c if cfg.enable_dr else None
        return out


# --------------------------------------------------------------------------
# Verification attention: each tree token attends to the prefix and to its
# ancestors-and-self only (Section "Tree Reranking Phase", last paragraph).
# --------------------------------------------------------------------------
def _gather_kv(cache, b, npos, page_size, page_table):
    """Rows 0..npos-1 of sequence b: [npos, Hkv, D]."""
    if page_size == 0:
        return cache[b, :npos]
    pos = np.arange(npos)
    pages = page_table[b, pos // page_size]
    return cache[pages, pos % page_size]


def tree_attention(q, k_cache, v_cache, page_size, page_table, kv_len, anc, n_tree, scale=None, only=None):
    """out[b,t,h] = softmax_p(q.k_p * scale) . v_p over p in [0, L_b) and the
    tree positions L_b + j for every j set in anc[b,t].  Rows t >= n_tree[b] are
    not part of the result (returned as zeros).  q: [B, Ncap, Hq, D]; paged caches [num_pages, page, Hkv, D] or
    contiguous [B, Lmax, Hkv, D] (page_size 0); all float64.  `only`: optional
    set of (b, t, h) to compute (the other entries stay zero) - for sampled
    checks at sizes where the full loop would take minutes."""
    B, Ncap, Hq, D = q.shape
    Hkv = k_cache.shape[-2]
    G = Hq // Hkv
    if scale is None or scale == 0:
        scale = 1.0 / np.sqrt(D)
    out = np.zeros_like(q, dtype=np.float64)
    for b in range(B):
        L, N = int(kv_len[b]), int(n_tree[b])
        if only is not None and not any(o[0] == b for o in only):
            continue
        Kb = np.asarray(_gather_kv(k_cache, b, L + N, page_size, page_table), dtype=np.float64)
        Vb = np.asarray(_gather_kv(v_cache, b, L + N, page_size, page_table), dtype=np.float64)
        for t in range(N):
            bits = [j for j in range(N) if (int(anc[b, t, j // 32]) >> (j % 32)) & 1]
            vis = np.concatenate([np.arange(L), L + np.array(bits, dtype=np.int64)]).astype(np.int64)
            for h in range(Hq):
                if only is not None and (b, t, h) not in only:
                    continue
                kh = h // G
                s = (Kb[vis, kh] @ np.asarray(q[b, t, h], dtype=np.float64)) * scale
                w = np.exp(s - np.max(s))
                w = w / np.sum(w)
                out[b, t, h] = w @ Vb[vis, kh]
    return out


# --------------------------------------------------------------------------
# Greedy (temperature 0) acceptance: with a one-hot target distribution the
# rule u <= min(1, p/q) accepts a draft token iff it equals the target argmax.
# --------------------------------------------------------------------------
def greedy_accept(target_logits, tokens, parent, n_tree, max_depth):
    B = tokens.shape[0]
    accept_len = np.zeros((B,), dtype=np.int32)
    accept_path = np.full((B, max_depth + 1), -1, dtype=np.int32)
    bonus = np.zeros((B,), dtype=np.int32)
    for b in range(B):
        N = int(n_tree[b])
        g = [int(np.argmax(target_logits[b, t])) for t in range(N)]  # first maximum: lower id wins ties
        cur, path = 0, [0]
        while True:
            nxt = -1
            for c in range(N):
                if parent[b, c] == cur and tokens[b, c] == g[cur]:
                    nxt = c
                    break
            if nxt < 0:
                break
            cur = nxt
            path.append(cur)
        accept_len[b] = len(path) - 1
        accept_path[b, : len(path)] = path
        bonus[b] = g[cur]
    return accept_len, accept_path, bonus


# --------------------------------------------------------------------------
# Stochastic acceptance at temperature T > 0 (Section "Speculative Decoding").
# The paper states the rule for a chain: draft token x with q = P_D(x | .),
# p = P_T(x | .) and u ~ Uniform(0,1) is accepted iff u <= min(1, p/q);
# otherwise decoding falls back to a sample of norm(max(0, P_T - P_D)).
# Reading for a tree (the paper only says that the siblings of a rejected token
# stay in play): at a node the children are tried in tree order; after a
# rejection P_T is replaced by the residual norm(max(0, P_T - P_D)) and the next
# sibling is tried against that, P_D unchanged (children are draws from P_D);
# when no child is left the bonus token is drawn from the distribution that
# stands then - the target distribution at a leaf, a residual otherwise - by
# inversion of its cumulative sum in token order.  A residual that sums to zero
# (reachable only through a rejection of probability zero) ends the sibling
# loop with the distribution before it.
# The random numbers are inputs: u_accept[b, c] decides tree node c, u_bonus[b]
# draws the bonus token.
# Besides the results, the smallest distance of a decision from its threshold
# is returned (relative), so that a comparison with another implementation can
# tell a wrong result from a rounding-order coin flip.
# --------------------------------------------------------------------------
def _softmax_t(logits, T):
    s = np.asarray(logits, dtype=np.float64) / T
    e = np.exp(s - np.max(s))
    return e / np.sum(e)


def stochastic_accept(target_logits, draft_logits, tokens, parent, n_tree, max_depth, temperature, u_accept, u_bonus):
    B = tokens.shape[0]
    accept_len = np.zeros((B,), dtype=np.int32)
    accept_path = np.full((B, max_depth + 1), -1, dtype=np.int32)
    bonus = np.zeros((B,), dtype=np.int32)
    margin = np.full((B,), np.inf)
    for b in range(B):
        N = int(n_tree[b])
        cur, path = 0, [0]
        while True:
            p = _softmax_t(target_logits[b, cur], temperature)  # P_T(. | path to cur)
            children = [c for c in range(N) if parent[b, c] == cur]
            nxt = -1
            if children:
                q = _softmax_t(draft_logits[b, cur], temperature)  # P_D(. | path to cur)
                for c in children:
                    x = int(tokens[b, c])
                    ratio = min(1.0, p[x] / q[x]) if q[x] > 0.0 else 1.0
                    u = float(u_accept[b, c])
                    if ratio < 1.0:
                        margin[b] = min(margin[b], abs(u - ratio))
                    if u <= ratio:
                        nxt = c
                        break
                    residual = np.maximum(0.0, p - q)
                    total = np.sum(residual)
                    if not total > 0.0:
                        break
                    p = residual / total
            if nxt < 0:
                break
            cur = nxt
            path.append(cur)
        cdf = np.cumsum(p)
        goal = float(u_bonus[b]) * cdf[-1]
        x = int(np.argmax(cdf >= goal))  # first token whose cumulative sum reaches the goal
        below = cdf[x - 1] if x > 0 else 0.0
        margin[b] = min(margin[b], (cdf[x] - goal) / cdf[-1], (goal - below) / cdf[-1])
        accept_len[b] = len(path) - 1
        accept_path[b, : len(path)] = path
        bonus[b] = x
    return accept_len, accept_path, bonus, margin


# --------------------------------------------------------------------------
# KV compaction: the accepted nodes' cache rows become contiguous after the
# prefix.  The paper does not describe it; this is the plain gather.
# --------------------------------------------------------------------------
def compact_kv(k_cache, v_cache, page_size, page_table, kv_len, accept_path, accept_len):
    """Caches carry a leading layer axis: [n_layers, ...].  Returns new caches
    (copies) and the new kv_len = L_b + accept_len + 1."""
    newk, newv = k_cache.copy(), v_cache.copy()
    new_len = np.array(kv_len, dtype=np.int32).copy()

    def addr(b, pos):
        if page_size == 0:
            return (b, pos)
        return (int(page_table[b, pos // page_size]), pos % page_size)

    for b in range(len(kv_len)):
        L, a = int(kv_len[b]), int(accept_len[b])
        for j in range(a + 1):
            src = addr(b, L + int(accept_path[b, j]))
            dst = addr(b, L + j)
            for old, new in ((k_cache, newk), (v_cache, newv)):
                new[(slice(None),) + dst] = old[(slice(None),) + src]
        new_len[b] = L + a + 1
    return newk, newv, new_len
