"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types an oracle formula: each compares the oracle with a
hand-worked value, a closed form, an exact-arithmetic evaluation, a brute-force
enumeration or a separately coded textbook routine.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import (
    CastOracle,
    CostTable,
    OracleConfig,
    alg1_is_stable,
    alg1_select_max_valid_index,
    ancestor_masks,
    compact_kv,
    greedy_accept,
    log_sum_exp,
    select_grid,
    stochastic_accept,
    topk_children,
    tree_attention,
)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- Algorithm 1
def test_alg1_hand_worked_cases():
    for ln in _golden_lines("alg1_cases.txt"):
        C, u, c, marks, out = [p.strip() for p in ln.split("|")]
        u = [float(x) for x in u.split()]
        c = [float(x) for x in c.split()]
        assert alg1_select_max_valid_index(u, c, float(C)) == int(out), ln
        # the golden marks imply the output; check the file is self-consistent
        marks = [int(x) for x in marks.split()]
        assert max(j + 1 for j, mk in enumerate(marks) if mk) == int(out)


def test_alg1_equals_min_chord_slope_definition_exact():
    """mark[j] = 1 iff every chord from an earlier index has slope >= C; checked
    in exact rational arithmetic on random non-concave inputs."""
    rng = np.random.default_rng(7)
    for _ in range(200):
        n = int(rng.integers(1, 9))
        u = [Fraction(int(x), 16) for x in np.cumsum(rng.integers(0, 12, size=n))]
        c = [Fraction(int(x), 8) for x in np.cumsum(rng.integers(1, 6, size=n))]
        C = Fraction(int(rng.integers(1, 9)), 4)
        best = 1
        for j in range(1, n):
            if all((u[j] - u[i]) / (c[j] - c[i]) >= C for i in range(j)):
                best = j + 1
        assert alg1_select_max_valid_index(u, c, C) == best


def test_alg1_theorem_linear_cost_special_case_exact():
    """Theorem: c_j = lambda*j + delta and C1 = mean_b v^(b)(K) / lambda give
    output K (strictly decreasing batch-mean values), in exact arithmetic."""
    rng = np.random.default_rng(11)
    for trial in range(50):
        B = int(rng.integers(1, 4))
        n = int(rng.integers(2, 9))
        # per-row strictly decreasing dyadic values
        rows = []
        for _ in range(B):
            exps = np.sort(rng.choice(np.arange(1, 20), size=n, replace=False))
            rows.append([Fraction(1, 2 ** int(e)) for e in exps])
        lam, delta = Fraction(int(rng.integers(1, 9)), 100), Fraction(int(rng.integers(0, 5)), 7)
        u = [sum(sum(r[: k + 1]) for r in rows) / B for k in range(n)]  # Eq. 1
        c = [lam * (j + 1) + delta for j in range(n)]
        for K in range(1, n + 1):
            C1 = sum(r[K - 1] for r in rows) / (B * lam)
            assert alg1_select_max_valid_index(u, c, C1) == K


def test_alg1_theorem_tie_keeps_next_index():
    # v(K) == v(K+1): slope exactly C is not '< C', so K+1 survives.
    v = [Fraction(1, 2), Fraction(1, 4), Fraction(1, 4), Fraction(1, 8)]
    u = list(itertools.accumulate(v))
    c = [Fraction(j + 1) for j in range(4)]
    assert alg1_select_max_valid_index(u, c, v[1]) == 3


def test_alg1_stability_flag():
    u, c = [1.0, 2.0, 3.0], [1.0, 2.0, 3.0]
    assert not alg1_is_stable(u, c, 1.0)  # sits exactly on the boundary
    assert alg1_is_stable(u, c, 0.5)


# -------------------------------------------------------------------- select()
def test_select_grid_hand_table():
    for ln in _golden_lines("select_grid_cases.txt"):
        L, M, c, want = [int(x) for x in ln.split()]
        assert select_grid(c, L, M) * L == want, ln


# ------------------------------------------------------------- lse and top-K
def test_lse_normalises_and_uniform_closed_form():
    rng = np.random.default_rng(3)
    x = rng.normal(0, 3, size=5000)
    assert abs(np.sum(np.exp(x - log_sum_exp(x))) - 1.0) < 1e-12
    V = 4096
    assert abs(log_sum_exp(np.zeros(V)) - np.log(V)) < 1e-12
    assert abs(log_sum_exp(np.array([-np.inf, 0.0, -np.inf])) - 0.0) < 1e-15


def test_topk_ties_lower_token_first():
    x = np.array([1.0, 3.0, 3.0, -1.0, 3.0, 0.0, -0.0])
    assert list(topk_children(x, 4)) == [1, 2, 4, 0]
    assert list(topk_children(np.array([0.0, -0.0, 0.0]), 2)) == [0, 1]


def test_uniform_logits_children_have_logprob_minus_logV():
    V, K = 64, 3
    cfg = OracleConfig(vocab=V, top_k=K, max_depth=2, total_token=8, max_tree=32)
    o = CastOracle(cfg)
    o.step_begin([5], [10])
    o.expand(1, np.zeros((1, K, V)))
    o.expand(2, np.zeros((1, K, V)))
    assert np.allclose(o.score[0][1:4], -np.log(V), atol=1e-13)
    assert np.allclose(o.score[0][4:], -2 * np.log(V), atol=1e-13)
    assert o.token[0][1:4] == [0, 1, 2]


# ------------------------------------------- brute force on tiny vocabularies
def _path_logits(seed, V):
    """A deterministic 'draft model': logits as a function of the token path."""
    cache = {}

    def f(path):
        if path not in cache:
            r = np.random.default_rng([seed] + list(path) + [len(path)])
            cache[path] = r.normal(0, 1.5, size=V)
        return cache[path]

    return f


def _run_oracle_on_model(model, V, K, H, m, root=0, pool_mode=0):
    cfg = OracleConfig(vocab=V, top_k=K, max_depth=H, total_token=m, max_tree=32, pool_mode=pool_mode)
    o = CastOracle(cfg)
    o.step_begin([root], [0])

    def path_of(p):
        toks = []
        while p > 0:
            toks.append(o.token[0][p])
            p = o.parent[0][p]
        return tuple(reversed(toks))

    for layer in range(1, H + 1):
        logits = np.zeros((1, K, V))
        for r, p in enumerate(o.retained[0]):
            logits[0, r] = model(path_of(p))
        o.expand(layer, logits)
    return o, o.select_nodes(), path_of


@pytest.mark.parametrize("V,K,H,m", [(3, 2, 3, 5), (4, 2, 3, 7), (4, 2, 2, 4), (3, 1, 3, 3), (4, 2, 3, 11)])
def test_expansion_and_rerank_match_brute_force(V, K, H, m):
    for seed in range(6):
        model = _path_logits(seed, V)
        o, sel, path_of = _run_oracle_on_model(model, V, K, H, m)

        # brute force: value of every path by direct products of softmax probabilities
        def prob(path):
            v = 1.0
            for d in range(len(path)):
                x = model(path[:d])
                v *= np.exp(x[path[d]]) / np.sum(np.exp(x))
            return v

        # expansion: layer by layer, top-K children of each retained node, keep top-K by value
        retained = [()]
        pool = [()]
        for d in range(1, H + 1):
            cands = []
            for par in retained:
                x = model(par)
                kids = sorted(range(V), key=lambda t: (-x[t], t))[:K]
                cands += [par + (t,) for t in kids]
            pool += cands
            retained = sorted(cands, key=lambda p: -prob(p))[:K]
            got = [path_of(p) for p in o.retained[0]] if d == H else None
            if got is not None:
                assert got == retained
        assert sorted(path_of(p) for p in range(o.pool_size)) == sorted(pool)
        for p in range(o.pool_size):
            assert abs(np.exp(o.score[0][p]) - prob(path_of(p))) < 1e-12

        # rerank: the kept nodes are the top-N of the pool by value ...
        N = int(sel["n_tree"][0])
        assert N == min(len(pool), m)
        kept = {path_of(int(p)) for p in sel["pool_idx"][0, :N]}
        assert kept == set(sorted(pool, key=lambda p: -prob(p))[:N])
        # ... form a connected rooted subtree ...
        assert () in kept and all(p[:-1] in kept for p in kept if p)
        # ... and maximise the total value over ALL connected rooted subtrees of that size
        others = [p for p in pool if p]
        best = -1.0
        for sub in itertools.combinations(others, N - 1):
            s = set(sub) | {()}
            if all(p[:-1] in s for p in sub):
                best = max(best, sum(prob(p) for p in s))
        assert abs(sum(prob(p) for p in kept) - best) < 1e-12


def test_pool_mode_retained_only_is_subset_and_sized():
    V, K, H = 4, 2, 3
    model = _path_logits(5, V)
    o, sel, path_of = _run_oracle_on_model(model, V, K, H, m=32, pool_mode=1)
    N = int(sel["n_tree"][0])
    assert N == sum(o.n_hist)  # N = min(sum_i n_i, m) with the root as n_0 = 1
    assert all(o.kept_flag[0][int(p)] for p in sel["pool_idx"][0, :N])


# ------------------------------------------------------- invariants of a tree
def _random_tree_run(seed, B=3, V=50, K=3, H=4, m=20, **kw):
    rng = np.random.default_rng(seed)
    cfg = OracleConfig(vocab=V, top_k=K, max_depth=H, total_token=m, max_tree=32, **kw)
    tables = None
    if kw.get("enable_bp") or kw.get("enable_dp") or kw.get("enable_dr"):
        n = np.arange(1, 33, dtype=np.float64)[None, :]
        g = np.arange(1, 5, dtype=np.float64)[:, None]
        fT = 1.0 + 0.1 * g + 0.05 * n
        tables = {B: CostTable(B, 16, 4, 32, fT, 0.1 * fT)}
    o = CastOracle(cfg, tables)
    o.step_begin(rng.integers(0, V, size=B), rng.integers(1, 40, size=B))
    for layer in range(1, H + 1):
        o.expand(layer, rng.normal(0, 2, size=(B, K, V)))
    return o, o.select_nodes()


@pytest.mark.parametrize("kw", [{}, {"enable_bp": 1, "enable_dr": 1, "C1": 0.5, "C3": 0.2},
                                {"enable_bp": 1, "enable_dp": 1, "enable_dr": 1, "C1": 0.3, "C2": 0.5, "C3": 0.1},
                                {"pool_mode": 1}])
def test_tree_invariants(kw):
    for seed in range(5):
        o, sel = _random_tree_run(seed, **kw)
        cfg = o.cfg
        for i, n_i in enumerate(o.n_hist[1:], start=1):
            assert 1 <= n_i <= min(o.n_hist[i - 1] * cfg.top_k, cfg.width)
        for b in range(o.B):
            N = int(sel["n_tree"][b])
            assert 1 <= N <= cfg.total_token
            par, dep, tok, sc = sel["parent"][b], sel["depth"][b], sel["tokens"][b], sel["scores"][b]
            assert par[0] == -1 and dep[0] == 0 and sel["pool_idx"][b, 0] == 0
            for t in range(1, N):
                assert 0 <= par[t] < t
                assert dep[t] == dep[par[t]] + 1
                assert sc[t] <= sc[par[t]]
            for t in range(N):
                sib = [tok[c] for c in range(N) if par[c] == t]
                assert len(sib) == len(set(sib))
                want = sel["anc"][b, par[t]].copy() if par[t] >= 0 else np.zeros_like(sel["anc"][b, t])
                want[t // 32] |= np.uint32(1 << (t % 32))
                assert np.array_equal(sel["anc"][b, t], want)
            assert np.all(sel["tokens"][b, N:] == -1) and not sel["anc"][b, N:].any()


def test_all_switches_off_is_fixed_eagle2_mode():
    o, sel = _random_tree_run(1, B=2, K=3, H=4, m=20)
    assert o.n_hist == [1, 3, 3, 3, 3]
    assert o.pool_size == 1 + 3 + 3 * 9
    assert list(sel["n_tree"]) == [20, 20]


# -------------------------------------------------------------- depth pruning
def test_depth_pruning_scripted_fifo():
    """B=1, K=1 chain with dyadic probabilities: layer values 1/2, 1/4, 1/16, so
    phi_1 = 1/2 and phi_2 = 1/4 on every step; draft cost c_1 = 0.1, C2 = 1, R = 2.
    FIFO contents and the go/no-go decisions were worked by hand."""
    V, H = 4, 3
    ninf = -np.inf
    rows = {1: [0.0, 0.0, ninf, ninf], 2: [0.0, 0.0, ninf, ninf], 3: [0.0, 0.0, 0.0, 0.0]}
    cfg = OracleConfig(vocab=V, top_k=1, max_depth=H, total_token=8, max_tree=32, enable_dp=1, C2=1.0, fifo_len=2)
    tab = CostTable(1, 8, 2, 2, [[1.0, 2.0], [1.0, 2.0]], [[0.1, 0.2], [0.1, 0.2]])
    o = CastOracle(cfg, {1: tab})

    def step():
        o.step_begin([0], [3])
        return [o.expand(l, np.array(rows[l], dtype=np.float64).reshape(1, 1, V))[2] for l in (1, 2, 3)]

    # step 1: alpha_1 = 1 -> 0.5/0.1 = 5 >= 1; alpha_2 = 1 -> 0.25/0.1 = 2.5 >= 1
    assert step() == [1, 1, 0]
    assert np.allclose(o.fifo[0], [1, 0.5]) and np.allclose(o.fifo[1], [1, 0.25])
    # step 2: alpha_1 = 0.75 -> 3.75; A_1 evicts the initial 1; alpha_2 = 0.625 -> 1.5625 >= 1
    assert step() == [1, 1, 0]
    assert np.allclose(o.fifo[0], [0.5, 0.5]) and np.allclose(o.fifo[1], [0.25, 0.25])
    # step 3: alpha_1 = 0.5 -> 2.5 go; alpha_2 = 0.25 -> 0.625 < 1: layer 3 is not generated
    assert step() == [1, 0, 0]
    assert np.allclose(o.fifo[0], [0.5, 0.5]) and np.allclose(o.fifo[1], [0.25, 0.25])
    assert o.layers_done == 2 and o.pool_size == 3
    sel = o.select_nodes()
    assert int(sel["n_tree"][0]) == 3 and list(sel["parent"][0, :3]) == [-1, 0, 1]


# ------------------------------------------------------------------ attention
def _rand_attn_case(rng, B=2, N=6, Hq=4, Hkv=2, D=8, Lmax=9, page=0):
    kv_len = rng.integers(0, Lmax + 1, size=B)
    q = rng.normal(size=(B, 8, Hq, D))
    if page:
        per = (Lmax + 8 + page - 1) // page
        table = rng.permutation(per * B).reshape(B, per).astype(np.int32)
        shape = (per * B, page, Hkv, D)
    else:
        table, shape = None, (B, Lmax + 8, Hkv, D)
    k, v = rng.normal(size=shape), rng.normal(size=shape)
    return kv_len, q, k, v, table


def _seq_rows(cache, table, page, b, n):
    if page == 0:
        return cache[b, :n]
    return np.stack([cache[table[b, p // page], p % page] for p in range(n)])


def _dense_softmax_attention(q, K, V, scale):
    s = K @ q * scale
    w = np.exp(s - s.max())
    return (w / w.sum()) @ V


@pytest.mark.parametrize("page", [0, 4])
def test_attention_chain_tree_is_causal_attention(page):
    rng = np.random.default_rng(21)
    B, N, Hq, Hkv, D = 2, 6, 4, 2, 8
    kv_len, q, k, v, table = _rand_attn_case(rng, page=page)
    parent = np.array([-1, 0, 1, 2, 3, 4])
    anc = np.stack([ancestor_masks(parent, N, 1)] * B)
    anc = np.pad(anc, ((0, 0), (0, 2), (0, 0)))
    out = tree_attention(q, k, v, page, table, kv_len, anc, np.full(B, N), None)
    for b in range(B):
        L = int(kv_len[b])
        Kb, Vb = _seq_rows(k, table, page, b, L + N), _seq_rows(v, table, page, b, L + N)
        for h in range(Hq):
            # textbook causal attention: triangular mask over the L+N positions, queries at the last N
            S = (q[b, :N, h] @ Kb[:, h // 2].T) / np.sqrt(D)
            mask = np.tril(np.ones((L + N, L + N)))[L:]
            S = np.where(mask > 0, S, -np.inf)
            Wt = np.exp(S - S.max(axis=1, keepdims=True))
            Wt /= Wt.sum(axis=1, keepdims=True)
            assert np.allclose(out[b, :N, h], Wt @ Vb[:, h // 2], atol=1e-12)
    assert not out[:, N:].any()


def test_attention_each_node_equals_dense_attention_over_its_path():
    rng = np.random.default_rng(22)
    B, N, Hq, Hkv, D = 2, 7, 4, 2, 8
    kv_len, q, k, v, table = _rand_attn_case(rng, N=N, page=4)
    parent = np.array([-1, 0, 0, 1, 1, 2, 4])
    anc = np.pad(np.stack([ancestor_masks(parent, N, 1)] * B), ((0, 0), (0, 1), (0, 0)))
    out = tree_attention(q, k, v, 4, table, kv_len, anc, np.full(B, N), 0.37)
    for b in range(B):
        L = int(kv_len[b])
        Kb, Vb = _seq_rows(k, table, 4, b, L + N), _seq_rows(v, table, 4, b, L + N)
        for t in range(N):
            path, a = [], t
            while a >= 0:  # explicit walk to the root
                path.append(a)
                a = parent[a]
            idx = list(range(L)) + [L + j for j in reversed(path)]
            for h in range(Hq):
                want = _dense_softmax_attention(q[b, t, h], Kb[idx, h // 2], Vb[idx, h // 2], 0.37)
                assert np.allclose(out[b, t, h], want, atol=1e-12)


def test_attention_star_tree_equal_keys_and_empty_prefix():
    rng = np.random.default_rng(23)
    B, N, Hq, Hkv, D = 1, 5, 2, 1, 4
    q = rng.normal(size=(B, N, Hq, D))
    k = np.ones((B, 12, Hkv, D)) * 0.3  # all keys equal -> uniform weights
    v = rng.normal(size=(B, 12, Hkv, D))
    parent = np.array([-1, 0, 0, 0, 0])
    anc = ancestor_masks(parent, N, 1)[None]
    for L in (0, 6):
        out = tree_attention(q, k, v, 0, None, np.array([L]), anc, np.array([N]), None)
        for t in range(N):
            vis = list(range(L)) + sorted({L, L + t})
            want = v[0, vis, 0].mean(axis=0)  # closed form: mean of V over prefix + root + self
            assert np.allclose(out[0, t, 0], want, atol=1e-13)
            assert np.allclose(out[0, t, 1], want, atol=1e-13)


# --------------------------------------------------------------------- accept
def test_greedy_accept_equals_sequential_decoding():
    rng = np.random.default_rng(31)
    V, H = 11, 5
    for trial in range(40):
        N = int(rng.integers(1, 16))
        parent = np.array([-1] + [int(rng.integers(0, t)) for t in range(1, N)])
        depth = np.zeros(N, dtype=int)
        tokens = np.zeros(N, dtype=np.int32)
        tokens[0] = rng.integers(0, V)
        for t in range(1, N):
            depth[t] = depth[parent[t]] + 1
            used = {tokens[c] for c in range(1, t) if parent[c] == parent[t]}
            tokens[t] = rng.choice([x for x in range(V) if x not in used])
        if depth.max() > H:
            continue

        # a synthetic target "model": next token as a function of the token path so far
        def target_next(path_tokens):
            r = np.random.default_rng([trial, len(path_tokens)] + [int(x) for x in path_tokens])
            kids_bias = r.integers(0, V)
            return int(kids_bias)

        def tok_path(t):
            p = []
            while t >= 0:
                p.append(int(tokens[t]))
                t = parent[t]
            return tuple(reversed(p))

        # make roughly half of the decodes hit a child so that paths are non-trivial
        logits = rng.normal(size=(1, 16, V))
        want_next = {}
        for t in range(N):
            kids = [c for c in range(N) if parent[c] == t]
            nxt = target_next(tok_path(t))
            if kids and rng.random() < 0.6:
                nxt = int(tokens[kids[int(rng.integers(0, len(kids)))]])
            want_next[tok_path(t)] = nxt
            logits[0, t, nxt] = logits[0, t].max() + 1.0
        # sequential token-by-token decoding with the target, following the draft tree
        seq, cur = [int(tokens[0])], 0
        steps = 0
        while True:
            nxt = want_next[tuple(seq)]
            child = [c for c in range(N) if parent[c] == cur and tokens[c] == nxt]
            if not child:
                bonus = nxt
                break
            cur = child[0]
            seq.append(nxt)
            steps += 1
        al, ap, bo = greedy_accept(logits, tokens[None], parent[None], np.array([N]), H)
        assert al[0] == steps and bo[0] == bonus
        assert tuple(int(tokens[i]) for i in ap[0, : steps + 1]) == tuple(seq)
        assert np.all(ap[0, steps + 1:] == -1)


def test_greedy_accept_edge_cases():
    tokens = np.array([[7, 3, 4, 5, 6]], dtype=np.int32)
    parent = np.array([[-1, 0, 0, 2, 3]])
    logits = np.zeros((1, 5, 10))
    # no child matches: length 0, bonus = argmax at the root (ties -> lower id)
    al, ap, bo = greedy_accept(logits, tokens, parent, np.array([5]), 4)
    assert (al[0], bo[0], list(ap[0])) == (0, 0, [0, -1, -1, -1, -1])
    # match at a non-first sibling, then full-depth accept
    logits[0, 0, 4] = 1; logits[0, 2, 5] = 1; logits[0, 3, 6] = 1; logits[0, 4, 9] = 1
    al, ap, bo = greedy_accept(logits, tokens, parent, np.array([5]), 4)
    assert (al[0], bo[0], list(ap[0])) == (3, 9, [0, 2, 3, 4, -1])
    # nodes beyond n_tree are invisible
    al, ap, bo = greedy_accept(logits, tokens, parent, np.array([3]), 4)
    assert (al[0], bo[0]) == (1, 5)


def test_rerank_per_row_equals_independent_single_sequence_runs():
    """With the per-layer sizing off the expansion of a sequence does not depend on its batch, so a
    batch reranked per sequence must give every sequence the tree it gets when run alone with the same
    cost row (same table, same padded context); with one sequence the two modes coincide."""
    rng = np.random.default_rng(21)
    V, K, H, m, B = 40, 3, 3, 24, 4
    L, M, Ntab = 64, 4, 32
    fT = 1.0 + 0.03 * np.arange(1, Ntab + 1)[None, :] * np.ones((M, 1)) + 0.1 * np.arange(M)[:, None]
    fD = 0.05 * fT
    kw = dict(vocab=V, top_k=K, max_depth=H, total_token=m, max_tree=32, enable_dr=1, C3=0.6)
    root = rng.integers(0, V, size=B)
    kv = np.array([100, 100, 100, 100])
    logits = [rng.normal(size=(B, K, V)) * (1.0 + np.arange(B))[:, None, None] for _ in range(H)]  # sharper rows further down
    tabs = {B: CostTable(B, L, M, Ntab, fT, fD), 1: CostTable(1, L, M, Ntab, fT, fD)}

    def run(cfg_over, rows):
        o = CastOracle(OracleConfig(**kw, **cfg_over), tabs)
        o.step_begin(root[rows], kv[rows])
        for i in range(H):
            o.expand(i + 1, logits[i][rows])
        return o.select_nodes()

    batch = run(dict(rerank_per_row=1), np.arange(B))
    mean = run(dict(rerank_per_row=0), np.arange(B))
    assert len(set(int(x) for x in mean["n_tree"])) == 1
    assert len(set(int(x) for x in batch["n_tree"])) > 1  # the recipe does give ragged sizes
    for b in range(B):
        for mode in (0, 1):
            solo = run(dict(rerank_per_row=mode), np.array([b]))
            assert solo["n_tree"][0] == batch["n_tree"][b]
            for key in ("tokens", "parent", "depth", "pool_idx"):
                assert np.array_equal(solo[key][0], batch[key][b]), (b, key)
            assert np.array_equal(solo["anc"][0], batch["anc"][b])


# ------------------------------------------------------ stochastic acceptance
def test_stochastic_accept_hand_worked_chain_and_sibling():
    """P_T = (0.5, 0.3, 0.2), P_D = (0.2, 0.5, 0.3) at the root. A child with token 1 is accepted iff
    u <= 0.3/0.5; after its rejection the residual is norm(max(0, P_T - P_D)) = (1, 0, 0): a sibling
    with token 0 is then accepted for every u (ratio 1/0.2 > 1), one with token 2 never, and a bonus
    token drawn there is token 0 for every u."""
    lt = np.log(np.array([0.5, 0.3, 0.2]))
    ld = np.log(np.array([0.2, 0.5, 0.3]))
    leaf = np.log(np.array([0.1, 0.2, 0.7]))  # target distribution at every non-root node
    T = 1.0
    tl = np.stack([lt, leaf, leaf, leaf])[None]
    dl = np.stack([ld, ld, ld, ld])[None]

    def run(tokens, parent, ua, ub):
        al, ap, bo, _ = stochastic_accept(tl, dl, np.array([tokens], dtype=np.int32), np.array([parent]),
                                          np.array([len(tokens)]), 3, T, np.array([ua]), np.array([ub]))
        return int(al[0]), [int(x) for x in ap[0]], int(bo[0])

    # chain root -> token 1: accepted just below the ratio 0.6, bonus from the leaf's (0.1, 0.2, 0.7) by inversion
    assert run([9, 1], [-1, 0], [0.0, 0.59], 0.05) == (1, [0, 1, -1, -1], 0)
    assert run([9, 1], [-1, 0], [0.0, 0.59], 0.25) == (1, [0, 1, -1, -1], 1)
    assert run([9, 1], [-1, 0], [0.0, 0.59], 0.31) == (1, [0, 1, -1, -1], 2)
    # rejected just above it: bonus from the residual (1, 0, 0)
    for ub in (0.01, 0.5, 0.99):
        assert run([9, 1], [-1, 0], [0.0, 0.61], ub) == (0, [0, -1, -1, -1], 0)
    # siblings in tree order: token 1 rejected, then token 2 (residual probability 0) rejected, then token 0 accepted
    assert run([9, 1, 2, 0], [-1, 0, 0, 0], [0.0, 0.7, 1e-9, 0.999], 0.95) == (1, [0, 3, -1, -1], 2)
    # the uniform number of a node is used for that node only: token 0 first is accepted outright (ratio 2.5)
    assert run([9, 0, 1], [-1, 0, 0], [0.0, 0.999, 0.0], 0.0001) == (1, [0, 1, -1, -1], 0)
    # temperature: at T = 2 the root distributions are norm(sqrt(.)); token 1's ratio becomes
    # sqrt(0.3)/sum_T over sqrt(0.5)/sum_D
    sT, sD = np.sqrt([0.5, 0.3, 0.2]).sum(), np.sqrt([0.2, 0.5, 0.3]).sum()
    ratio = (np.sqrt(0.3) / sT) / (np.sqrt(0.5) / sD)
    for du, want in ((-1e-6, 1), (1e-6, 0)):
        al, _, _, mg = stochastic_accept(tl, dl, np.array([[9, 1]], dtype=np.int32), np.array([[-1, 0]]), np.array([2]), 3,
                                         2.0, np.array([[0.0, ratio + du]]), np.array([0.5]))
        assert al[0] == want and mg[0] < 2e-6


def test_stochastic_accept_one_hot_target_is_the_greedy_rule():
    rng = np.random.default_rng(5)
    V, H = 13, 6
    for trial in range(60):
        N = int(rng.integers(1, 20))
        parent = np.array([-1] + [int(rng.integers(0, t)) for t in range(1, N)])
        depth = np.zeros(N, dtype=int)
        for t in range(1, N):
            depth[t] = depth[parent[t]] + 1
        if depth.max() > H:
            continue
        tokens = rng.integers(0, V, size=N).astype(np.int32)
        tl = rng.normal(size=(1, N, V))
        for t in range(N):  # a one-hot target: one logit far above the rest; often a child's token
            kids = [c for c in range(N) if parent[c] == t]
            x = int(tokens[kids[int(rng.integers(0, len(kids)))]]) if kids and rng.random() < 0.7 else int(rng.integers(0, V))
            tl[0, t, x] = 5000.0
        dl = rng.normal(size=(1, N, V))
        ua, ub = rng.uniform(1e-6, 1 - 1e-6, size=(1, N)), rng.uniform(1e-6, 1 - 1e-6, size=(1,))
        got = stochastic_accept(tl, dl, tokens[None], parent[None], np.array([N]), H, 1.0, ua, ub)
        want = greedy_accept(tl, tokens[None], parent[None], np.array([N]), H)
        # duplicate sibling tokens: the greedy walk takes the first match, and so does the stochastic one
        assert got[0][0] == want[0][0] and list(got[1][0]) == list(want[1][0]) and got[2][0] == want[2][0]


def test_stochastic_accept_equal_models_accept_every_first_child():
    rng = np.random.default_rng(6)
    V, N = 50, 9
    parent = np.array([[-1, 0, 0, 1, 1, 3, 2, 5, 5]])
    tokens = rng.integers(0, V, size=(1, N)).astype(np.int32)
    tl = rng.normal(size=(1, N, V)) * 2
    for T in (1.0, 0.5):
        ua, ub = rng.uniform(size=(1, N)), rng.uniform(size=(1,))
        al, ap, bo, _ = stochastic_accept(tl, tl.copy(), tokens, parent, np.array([N]), 5, T, ua, ub)
        assert al[0] == 4 and list(ap[0]) == [0, 1, 3, 5, 7, -1]
        # the bonus token: inversion of the leaf's distribution by a library routine
        z = tl[0, 7] / T
        pr = np.exp(z - z.max())
        cdf = np.cumsum(pr / pr.sum())
        assert bo[0] == int(np.searchsorted(cdf, ub[0] * cdf[-1], side="left"))


def test_stochastic_accept_output_follows_the_target_distribution():
    """With children drawn independently from P_D, the token the step emits at a node - an accepted
    child's or the bonus token - is distributed exactly as P_T at that node, whatever P_D is. Checked
    by simulation on a two-level tree over a 4-token vocabulary: first emitted token against
    P_T(. | root), second against P_T(. | first) given that the first was an accepted child."""
    rng = np.random.default_rng(11)
    V, trials = 4, 24000
    PT0, PD0 = np.array([0.45, 0.05, 0.2, 0.3]), np.array([0.1, 0.4, 0.3, 0.2])
    PT1 = rng.dirichlet(np.ones(V), size=V)  # P_T(. | first token)
    PD1 = rng.dirichlet(np.ones(V), size=V)
    first = np.zeros(V)
    second = np.zeros((V, V))
    for _ in range(trials):
        kids = rng.choice(V, size=3, p=PD0)
        tokens = [0] + [int(x) for x in kids]
        parent = [-1, 0, 0, 0]
        for c in (1, 2, 3):
            g = rng.choice(V, size=2, p=PD1[tokens[c]])
            tokens += [int(x) for x in g]
            parent += [c, c]
        N = len(tokens)
        tl = np.zeros((1, N, V))
        dl = np.zeros((1, N, V))
        tl[0, 0], dl[0, 0] = np.log(PT0), np.log(PD0)
        for c in (1, 2, 3):
            tl[0, c], dl[0, c] = np.log(PT1[tokens[c]]), np.log(PD1[tokens[c]])
        for c in range(4, N):
            tl[0, c] = np.log(PT0)  # never sampled from in what is counted below
        al, ap, bo, _ = stochastic_accept(tl, dl, np.array([tokens], dtype=np.int32), np.array([parent]), np.array([N]), 3, 1.0,
                                          rng.uniform(size=(1, N)), rng.uniform(size=(1,)))
        out = [tokens[i] for i in ap[0, 1: al[0] + 1]] + [int(bo[0])]
        first[out[0]] += 1
        if al[0] >= 1:
            second[out[0], out[1]] += 1
    assert np.all(np.abs(first / trials - PT0) < 5 * np.sqrt(PT0 * (1 - PT0) / trials))
    for x in range(V):
        n = second[x].sum()
        assert n > 500
        assert np.all(np.abs(second[x] / n - PT1[x]) < 5 * np.sqrt(PT1[x] * (1 - PT1[x]) / n) + 1e-9)


# ----------------------------------------------------------------- compaction
@pytest.mark.parametrize("page", [0, 4])
def test_compaction_is_an_out_of_place_gather(page):
    rng = np.random.default_rng(41)
    B, Hkv, D, nl = 2, 2, 4, 3
    kv_len = np.array([5, 9])
    per = 6
    if page:
        table = rng.permutation(per * B).reshape(B, per).astype(np.int32)
        shape = (nl, per * B, page, Hkv, D)
    else:
        table, shape = None, (nl, B, 24, Hkv, D)
    k, v = rng.normal(size=shape), rng.normal(size=shape)
    path = np.array([[0, 2, 3, -1], [0, 1, 2, 3]])  # row 0 overlaps: slot 2 is both a destination and a source
    alen = np.array([2, 3])
    nk, nv, nlen = compact_kv(k, v, page, table, kv_len, path, alen)
    assert list(nlen) == [8, 13]

    def row(c, l, b, pos):
        return c[l, b, pos] if page == 0 else c[l, table[b, pos // page], pos % page]

    for l in range(nl):
        for b in range(B):
            L = kv_len[b]
            for pos in range(L):  # prefix untouched
                assert np.array_equal(row(nk, l, b, pos), row(k, l, b, pos))
            for j in range(alen[b] + 1):
                assert np.array_equal(row(nk, l, b, L + j), row(k, l, b, L + path[b, j]))
                assert np.array_equal(row(nv, l, b, L + j), row(v, l, b, L + path[b, j]))
    # identity path leaves the cache as it was
    nk2, _, _ = compact_kv(k, v, page, table, kv_len, np.array([[0, 1, 2, 3]] * 2), np.array([3, 3]))
    assert np.array_equal(nk2, k)


# ------------------------------------- hand-worked steps with the sizing switches on
def _close(got, want_fracs, tol=1e-12):
    want = np.array([float(v) for v in want_fracs])
    got = np.asarray(got, dtype=np.float64)
    return got.shape == want.shape and bool(np.all(np.abs(got - want) <= tol * np.maximum(1.0, np.abs(want))))


def _run_golden_case(case):
    """Feeds a hand-worked case to the oracle and checks every written-out value."""
    import golden_cases  # noqa: F401  (tests/ is on sys.path under pytest)

    tables = None
    if case.fT:
        L, M, Ntab, fT, fD = case.table_arrays()
        tables = {case.B: CostTable(case.B, L, M, Ntab, fT, fD)}
    o = CastOracle(OracleConfig(**case.config_kwargs()), tables)
    H = int(case.param["H"])
    for step in case.steps():
        o.step_begin(case.root, case.kv_len)
        for layer in range(1, H + 1):
            nt, npr, cnt = o.expand(layer, case.logits(layer))
            if layer not in case.layers(step):
                assert cnt == 0 and o.layers_done < layer, f"step {step}: layer {layer} should not exist"
                continue
            key = ("step", step, "layer", layer)
            n_i = case.ints(*key, "n")[0][0]
            assert o.n_hist[layer] == n_i, (key, o.n_hist)
            assert cnt == case.ints(*key, "next_count")[0][0], (key, cnt)
            if case.has(*key, "u"):
                assert _close(o.last_u, case.get(*key, "u")[0]), (key, o.last_u)
            if case.has(*key, "c"):
                assert _close(o.last_c, case.get(*key, "c")[0]), (key, o.last_c)
            for b in range(case.B):
                assert list(nt[b, :n_i]) == case.ints(*key, "next_tokens")[b], (key, b, nt[b])
                assert list(npr[b, :n_i]) == case.ints(*key, "next_parent_row")[b], (key, b, npr[b])
        if case.has("step", step, "fifo"):
            for i, want in enumerate(case.get("step", step, "fifo")):
                assert _close(o.fifo[i], want), (step, i, o.fifo[i])
        if case.has("step", step, "N"):
            sel = o.select_nodes()
            _check_selection(case, ("step", step), sel, o)
    # the same expansion reranked under other budgets m (fixed-mode cases)
    for m in case.select_budgets():
        o.cfg.total_token = m
        _check_selection(case, ("select", "m", m), o.select_nodes(), o)


def _check_selection(case, key, sel, o):
    N = case.ints(*key, "N")[0][0]
    assert list(sel["n_tree"]) == [N] * case.B, (key, sel["n_tree"])
    if case.has(*key, "rerank", "u"):
        assert _close(o.last_u_sel, case.get(*key, "rerank", "u")[0]), (key, o.last_u_sel)
        assert _close(o.last_c_sel, case.get(*key, "rerank", "c")[0]), (key, o.last_c_sel)
    for name in ("tokens", "parent", "depth", "pool_idx"):
        for b in range(case.B):
            assert list(sel[name][b, :N]) == case.ints(*key, name)[b], (key, name, b, sel[name][b])
    if case.has(*key, "anc"):
        for b in range(case.B):
            assert list(sel["anc"][b, :N, 0]) == case.ints(*key, "anc")[b], (key, "anc", b)


def test_hand_worked_step_batch_two_all_switches():
    """Eq. 1 (batch mean of per-sequence prefix sums), Eq. 2 (draft row over the
    target's first entry, context = nodes retained so far), Algorithm 1 with C1,
    the depth test on c_{n_i} and the rerank (target row at n_0 = longest prefix,
    C3) composed as the paper states them: every intermediate value of two
    consecutive steps is compared with the hand derivation in the golden file."""
    import golden_cases

    (case,) = golden_cases.load("cast_step_b2.txt")
    _run_golden_case(case)


def test_hand_worked_exact_ties():
    """Order of exactly equal values (token id within a layer; depth first over
    the whole tree, so that the kept set is a tree) and the '>=' of the depth
    test at exact equality."""
    import golden_cases

    cases = golden_cases.load("cast_step_ties.txt")
    assert [c.name for c in cases] == ["layer_and_global_order", "depth_test_equality"]
    # the construction relies on these two floating-point facts
    assert np.log(0.5) + np.log(2.0) == 0.0 and np.exp(golden_cases.ZERO_PROB_LOGIT) == 0.0
    for case in cases:
        _run_golden_case(case)
