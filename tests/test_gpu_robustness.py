"""More parity through the C-ABI, beyond the hand-picked cases of test_gpu_parity.py:

* many small configurations drawn from fixed seeds (vocabulary sizes that are not multiples of
  anything, every K and W up to the caps, batch sizes, logit dtypes, the sizing switches, window starts,
  head groupings, random trees with shared sibling tokens), each compared with the oracle;
* the tree build at the hyper-parameters the paper reports for its own runs;
* one whole step with sentinel bands around every tensor the library writes."""
import numpy as np
import pytest
import torch

from oracle import CostTable, ancestor_masks, tree_attention
from paper_2510_26577_b200 import workloads as wl

from helpers import (assert_tree_equal, attention_tolerance, cfg_kwargs, gpu_attention, gpu_tree, make_tables, oracle_tree,
                     to_f64)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2510_26577_b200 import build
    build.build()
    from paper_2510_26577_b200 import binding as b
    b.load_library()
    return b


@pytest.mark.parametrize("seed", [1, 2])
def test_tree_build_random_configurations(binding, seed):
    rng = np.random.default_rng(seed)
    compared = 0
    for case in range(40):
        K, H = int(rng.integers(1, 17)), int(rng.integers(1, 5))
        B = int(rng.choice([1, 1, 2, 3, 5, 8, 16]))
        V = int(rng.choice([rng.integers(max(K, 17), 3000), rng.integers(3000, 40000), rng.integers(40000, 300000)]))
        while B * K * V * H > 3e7:  # keeps the oracle's sorts to seconds
            V = max(K + 1, V // 2)
        W = int(rng.integers(1, 17)) if rng.random() < 0.5 else 0
        m = int(rng.integers(2, 129))
        dt = "bf16" if rng.random() < 0.4 else "f32"
        cost = bool(rng.random() < 0.5)
        std = float(rng.choice([0.5, 2.0, 3.0]))
        w = wl.Workload("fuzz", 200 + case, B, "f32", dt, 4, 2, 64, 5, 600, 0, V, std, H, K, m, cost, 1, max_tree=128,
                        seed_salt=int(rng.integers(0, 50)))
        over = dict(max_width=W)
        if cost:
            over.update(enable_dp=int(rng.random() < 0.5), pool_mode=int(rng.random() < 0.3),
                        rerank_per_row=int(rng.random() < 0.3))
        kw = cfg_kwargs(w, **over)
        tables = raw = None
        if kw.get("enable_bp") or kw.get("enable_dp") or kw.get("enable_dr"):
            L, M, Ntab, fT, fD = make_tables(w, B)
            tables, raw = {B: CostTable(B, L, M, Ntab, fT, fD)}, (L, M, Ntab, fT, fD)
        ctx = binding.CastContext(max_batch=B, **kw)
        if raw:
            ctx.cast_set_cost_tables(B, *raw)
        root, kv = wl.root_tokens(w, "cpu").cuda(), wl.kv_lengths(w, "cpu").cuda()
        logits = [wl.draft_logits(w, l, "cpu", peaked=bool(case % 2), width=W).cuda() for l in range(1, H + 1)]
        o = oracle_tree(kw, tables, root, kv, logits)
        g = gpu_tree(ctx, root, kv, logits)
        assert ctx.cast_poll_status()[0] == 0, (case, kw)
        ctx.close()
        if o["min_score_gap"] < 1e-5 or not o["stable"]:
            continue  # a draw within rounding of a decision threshold proves nothing either way
        assert_tree_equal(g, o)
        compared += 1
    assert compared >= 28


def _random_parents(rng, N):
    return np.array([-1] + [int(rng.integers(max(0, t - 9), t)) for t in range(1, N)])


@pytest.mark.parametrize("seed", [3, 4, 5])
def test_attention_random_shapes_and_windows(binding, seed):
    rng = np.random.default_rng(seed)
    for case in range(24):
        dtype = "bf16" if rng.random() < 0.7 else "f32"
        D = int(rng.choice([64, 128]))
        Hkv = int(rng.choice([1, 2, 4, 8]))
        G = int(rng.choice([1, 2, 4, 7, 8]))
        Hq = Hkv * G
        page = int(rng.choice([0, 16]))
        B = int(rng.integers(1, 6))
        hi = int(rng.choice([40, 300, 1500]))
        w = wl.Workload("fuzz", 300 + case, B, dtype, "f32", Hq, Hkv, D, 0, hi, page, 100, 1.0, 4, 2, 8, False, 1)
        ctx = binding.CastContext(max_batch=B, vocab=100, top_k=2, max_depth=8, total_token=128, max_tree=128)
        # one seed runs with the early reads on (every input here is uploaded by a host copy that has completed
        # before the call, which is what the promise asks for)
        ctx.cast_set_attention_early_reads(seed == 4)
        kv = wl.kv_lengths(w, "cpu").cuda()
        n_tree = rng.integers(1, 129, size=B).astype(np.int32)
        first = np.array([int(rng.integers(0, n + 1)) if rng.random() < 0.6 else 0 for n in n_tree], dtype=np.int32)
        anc = np.zeros((B, 128, 4), dtype=np.uint32)
        for b in range(B):
            N = int(n_tree[b])
            anc[b, :N] = ancestor_masks(_random_parents(rng, N), N, 4)
        q = wl.query(w, 0, "cpu").cuda()
        k, v = (t.cuda() for t in wl.kv_cache(w, 0, "cpu"))
        table, num_pages = wl.page_table(w, "cuda")
        use_window = bool(first.any())
        out = gpu_attention(ctx, w, q, k, v, table, num_pages, kv, anc, torch.from_numpy(n_tree).cuda(),
                            first_row=torch.from_numpy(first).cuda() if use_window else None)
        assert ctx.cast_poll_status()[0] == 0
        got = to_f64(out)
        only = set()
        for b in range(B):
            lo, hi_t = (int(first[b]) if use_window else 0), int(n_tree[b])
            assert np.isnan(got[b, :lo]).all() and np.isnan(got[b, hi_t:]).all()
            assert np.isfinite(got[b, lo:hi_t]).all()
            if lo < hi_t:
                for t in {lo, hi_t - 1, int(rng.integers(lo, hi_t))}:
                    for h in {0, Hq - 1, int(rng.integers(0, Hq))}:
                        only.add((b, t, h))
        if not only:
            continue
        f32 = lambda t: t.float().cpu().numpy()
        tab = table.cpu().numpy() if table is not None else None
        ref = tree_attention(f32(q), f32(k), f32(v), page, tab, kv.cpu().numpy(), anc, n_tree, None, only)
        err = max(np.max(np.abs(got[i] - ref[i])) for i in only)
        assert err <= attention_tolerance(dtype), (case, dtype, D, Hq, Hkv, page, err)
        ctx.close()


@pytest.mark.parametrize("seed", [8, 9])
def test_attention_random_large_shapes(binding, seed):
    """bf16, D = 128, at sizes that reach every launch mode of the tensor-core kernel (clusters, the merge through
    a workspace, the plain launch): up to 48 ragged sequences, prefixes up to 20 000 positions (empty ones
    included), page sizes 0 / 16 / 64, group sizes that do and do not divide a row block, tree budgets 16 to 128
    with empty and full trees, early reads on for half of the cases. Rows past a tree stay untouched, live rows are
    finite, and sampled outputs of up to three sequences match the oracle."""
    rng = np.random.default_rng(seed)
    for case in range(14):
        D = 128
        Hkv = int(rng.choice([1, 2, 4, 8]))
        Hq = Hkv * int(rng.choice([1, 2, 4, 5, 8]))
        page = int(rng.choice([0, 16, 64]))
        B = int(rng.choice([1, 2, 3, 6, 12, 20, 33, 48]))
        hi = int(rng.choice([700, 3000, 9000, 20000]))
        while B * hi * Hkv * D > 1.2e8:  # keeps the cache to a few hundred MB and its generation to seconds
            if B > 1 and rng.random() < 0.5:
                B = max(1, B // 2)
            else:
                hi //= 2
        lo = int(rng.choice([0, hi // 2, hi]))
        Ncap = int(rng.choice([16, 64, 128]))
        w = wl.Workload("fuzz", 700 + case, B, "bf16", "f32", Hq, Hkv, D, lo, hi, page, 100, 1.0, 4, 2, 8, False, 1,
                        max_tree=Ncap)
        ctx = binding.CastContext(max_batch=B, vocab=100, top_k=2, max_depth=8, total_token=Ncap, max_tree=Ncap)
        ctx.cast_set_attention_early_reads(bool(rng.random() < 0.5))
        kv = wl.kv_lengths(w, "cpu").cuda()
        n_tree = rng.integers(0 if rng.random() < 0.2 else 1, Ncap + 1, size=B).astype(np.int32)
        if rng.random() < 0.3:
            n_tree[:] = Ncap
        anc = np.zeros((B, Ncap, ctx.words), dtype=np.uint32)
        for b in range(B):
            N = int(n_tree[b])
            if N:
                anc[b, :N] = ancestor_masks(_random_parents(rng, N), N, ctx.words)
        q = wl.query(w, 0, "cpu").cuda()
        k, v = (t.cuda() for t in wl.kv_cache(w, 0, "cpu"))
        table, num_pages = wl.page_table(w, "cuda")
        out = gpu_attention(ctx, w, q, k, v, table, num_pages, kv, anc, torch.from_numpy(n_tree).cuda())
        assert ctx.cast_poll_status()[0] == 0
        got = to_f64(out)
        only = set()
        for b in range(B):
            N = int(n_tree[b])
            assert np.isnan(got[b, N:]).all() and np.isfinite(got[b, :N]).all(), (case, b)
        for b in rng.choice(B, size=min(B, 3), replace=False):
            N = int(n_tree[b])
            if N:
                for t in {0, N - 1, int(rng.integers(0, N))}:
                    for h in {0, Hq - 1, int(rng.integers(0, Hq))}:
                        only.add((int(b), t, h))
        if only:
            f32 = lambda t: t.float().cpu().numpy()
            tab = table.cpu().numpy() if table is not None else None
            ref = tree_attention(f32(q), f32(k), f32(v), page, tab, kv.cpu().numpy(), anc, n_tree, None, only)
            err = max(np.max(np.abs(got[i] - ref[i])) for i in only)
            assert err <= attention_tolerance("bf16"), (case, B, Hq, Hkv, page, lo, hi, Ncap, err)
        ctx.close()


@pytest.mark.parametrize("seed", [6, 7])
def test_accept_and_compaction_random(binding, seed):
    from oracle import compact_kv, greedy_accept
    rng = np.random.default_rng(seed)
    for case in range(16):
        B, H = int(rng.integers(1, 7)), int(rng.integers(2, 9))
        Ncap = int(rng.choice([32, 64, 128]))
        V = int(rng.choice([rng.integers(50, 3000), rng.integers(3000, 70000)]))
        dt = "bf16" if rng.random() < 0.4 else "f32"
        page = int(rng.choice([0, 4, 16]))
        Hkv, D, n_layers = int(rng.choice([1, 2, 4])), int(rng.choice([64, 128])), int(rng.integers(1, 4))
        w = wl.Workload("fuzz", 400 + case, B, dt, dt, Hkv, Hkv, D, 3, 90, page, V, 2.0, H, 4, Ncap, False, n_layers,
                        max_tree=Ncap, seed_salt=seed)
        ctx = binding.CastContext(max_batch=B, vocab=V, top_k=4, max_depth=H, total_token=Ncap, max_tree=Ncap)
        n_tree = rng.integers(1, Ncap + 1, size=B).astype(np.int32)
        tokens = np.full((B, Ncap), -1, dtype=np.int32)
        parent = np.full((B, Ncap), -1, dtype=np.int32)
        for b in range(B):
            N = int(n_tree[b])
            par = _random_parents(rng, N)
            depth = np.zeros(N, dtype=int)
            for t in range(1, N):
                if depth[par[t]] + 1 > H:
                    par[t] = 0
                depth[t] = depth[par[t]] + 1
            parent[b, :N] = par
            tokens[b, :N] = rng.integers(0, V, size=N)  # siblings may share a token: the lowest index wins
        tl = wl.target_logits(w, "cpu")
        wl.plant_acceptance(w, tl, tokens, parent, n_tree)
        tl = tl.cuda()
        dev = lambda a: torch.from_numpy(a).cuda()
        alen = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        apath = torch.full((B, H + 1), -7, dtype=torch.int32, device="cuda")
        bonus = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        ctx.cast_accept(tl, B, dev(tokens), dev(parent), None, None, dev(n_tree), alen, apath, bonus)
        assert ctx.cast_poll_status()[0] == 0
        ol, op, ob = greedy_accept(to_f64(tl[:, : int(n_tree.max())]), tokens, parent, n_tree, H)
        assert np.array_equal(alen.cpu().numpy(), ol) and np.array_equal(apath.cpu().numpy(), op), case
        assert np.array_equal(bonus.cpu().numpy(), ob), case
        # compaction of all layers, compared as raw bits
        kv = wl.kv_lengths(w, "cpu").cuda()
        layers = [tuple(t.cuda() for t in wl.kv_cache(w, l, "cpu")) for l in range(n_layers)]
        kk = torch.stack([a for a, _ in layers]).contiguous()
        vv = torch.stack([c for _, c in layers]).contiguous()
        table, num_pages = wl.page_table(w, "cuda")
        bits = torch.int16 if dt == "bf16" else torch.int32
        k_old, v_old = kk.view(bits).cpu().numpy(), vv.view(bits).cpu().numpy()
        kv2 = kv.clone()
        ctx.cast_compact_kv(kk, vv, B, n_layers, kk[0].numel() * kk.element_size(), Hkv, D, page, table,
                            wl.seq_capacity(w) // (page or 1), num_pages, apath, alen, kv2)
        assert ctx.cast_poll_status()[0] == 0
        tab = table.cpu().numpy() if table is not None else None
        nk, nv, nlen = compact_kv(k_old, v_old, page, tab, kv.cpu().numpy(), op, ol)
        assert np.array_equal(kv2.cpu().numpy(), nlen), case
        assert np.array_equal(kk.view(bits).cpu().numpy(), nk) and np.array_equal(vv.view(bits).cpu().numpy(), nv), case
        ctx.close()


# ------------------------------------------------------------------ the paper's own hyper-parameters
@pytest.mark.parametrize("B,H,K,m,thr,V", [(1, 13, 12, 72, 3.5, 128256),   # batch 1: depth 13, top-k 12, 72 tokens
                                           (8, 9, 12, 72, 2.5, 32000)])    # batch 8: depth 9, top-k 12, 72 tokens
def test_tree_build_with_the_papers_settings(binding, B, H, K, m, thr, V):
    """Depth, top-k, token budget and threshold as the paper reports them for its runs (its one threshold
    is used for C1, C2 and C3), all three sizing switches on, peaked logits, two steps so that the
    depth-pruning buffers carry over."""
    w = wl.Workload("paper", 500 + B, B, "bf16", "f32", 32, 8, 128, 512, 2048, 16, V, 3.0, H, K, m, True, 1, max_tree=128)
    kw = cfg_kwargs(w, enable_dp=1, C1=thr, C2=thr, C3=thr)
    L, M, Ntab, fT, fD = make_tables(w, B)
    tables = {B: CostTable(B, L, M, Ntab, fT, fD)}
    ctx = binding.CastContext(max_batch=B, **kw)
    ctx.cast_set_cost_tables(B, L, M, Ntab, fT, fD)
    root, kv = wl.root_tokens(w, "cpu").cuda(), wl.kv_lengths(w, "cpu").cuda()
    oracle = None
    for step in range(2):
        logits = [wl.draft_logits(w, 20 * step + l, "cpu", peaked=True).cuda() for l in range(1, H + 1)]
        o = oracle_tree(kw, tables, root, kv, logits, oracle)
        oracle = o["oracle"]
        g = gpu_tree(ctx, root, kv, logits)
        assert ctx.cast_poll_status()[0] == 0
        assert o["min_score_gap"] >= 1e-5 and o["stable"], "a decision within rounding of its threshold: pick another seed"
        assert_tree_equal(g, o)
    assert 1 <= int(o["n_tree"][0]) <= m


# ------------------------------------------------------------------ nothing is written outside the outputs
class _Guarded:
    """Device buffers with a band of sentinel bytes on both sides of every output tensor."""
    BAND = 256  # bytes; a multiple of 16 so that the tensor inside keeps its alignment

    def __init__(self):
        self.items = []

    def alloc(self, shape, dtype, fill=None):
        n = int(np.prod(shape))
        size = torch.empty((), dtype=dtype).element_size()
        raw = torch.full((2 * self.BAND + n * size,), 0xA5, dtype=torch.uint8, device="cuda")
        inner = raw[self.BAND: self.BAND + n * size].view(dtype).view(*shape)
        if fill is not None:
            inner.fill_(fill)
        self.items.append(raw)
        return inner

    def check(self):
        for raw in self.items:
            assert bool((raw[: self.BAND] == 0xA5).all()) and bool((raw[-self.BAND:] == 0xA5).all())


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_guard_bands_around_every_output(binding, dtype):
    """One whole step (tree build, attention on the full tree and on a window, greedy and stochastic
    acceptance) with sentinel bands around every tensor the library writes: the bands stay intact and
    the results are the oracle's."""
    from oracle import greedy_accept
    B, H, K, m, Ncap = 3, 3, 4, 24, 32
    w = wl.Workload("guard", 600, B, dtype, "f32", 8, 2, 128 if dtype == "bf16" else 64, 100, 400, 16, 5000, 3.0, H, K, m, False,
                    1, max_tree=Ncap)
    kw = cfg_kwargs(w)
    ctx = binding.CastContext(max_batch=B, **kw)
    gd = _Guarded()
    root, kv = wl.root_tokens(w, "cpu").cuda(), wl.kv_lengths(w, "cpu").cuda()
    logits = [wl.draft_logits(w, l, "cpu").cuda() for l in range(1, H + 1)]
    ctx.cast_step_begin(B, root, kv)
    per_layer = []
    for i, lg in enumerate(logits, start=1):
        nt, npr, cnt = gd.alloc((B, K), torch.int32), gd.alloc((B, K), torch.int32), gd.alloc((1,), torch.int32)
        ctx.cast_tree_expand(i, lg, nt, npr, cnt)
        per_layer.append((nt, npr, cnt))
    tr = dict(tokens=gd.alloc((B, Ncap), torch.int32), parent=gd.alloc((B, Ncap), torch.int32),
              depth=gd.alloc((B, Ncap), torch.int32), anc=gd.alloc((B, Ncap, ctx.words), torch.int32),
              pool_idx=gd.alloc((B, Ncap), torch.int32), scores=gd.alloc((B, Ncap), torch.float64),
              n_tree=gd.alloc((B,), torch.int32))
    ctx.cast_select_nodes(tr["tokens"], tr["parent"], tr["depth"], tr["anc"], tr["pool_idx"], tr["scores"], tr["n_tree"])
    assert ctx.cast_poll_status()[0] == 0
    o = oracle_tree(kw, None, root, kv, logits)
    g = {k: v.cpu().numpy() for k, v in tr.items()}
    g["anc"] = g["anc"].view(np.uint32)
    g["per_layer"] = [(a.cpu().numpy(), b.cpu().numpy(), int(c.item())) for a, b, c in per_layer]
    g["status"], g["info"] = (0, 0), ctx.cast_step_info()
    assert_tree_equal(g, o)
    # attention: the whole tree, then a window
    q = wl.query(w, 0, "cpu").cuda()
    k, v = (t.cuda() for t in wl.kv_cache(w, 0, "cpu"))
    table, num_pages = wl.page_table(w, "cuda")
    seq_cap = wl.seq_capacity(w) // w.page_size
    tab = table.cpu().numpy()
    f32 = lambda t: t.float().cpu().numpy()
    ctx.cast_reserve_attention(q.dtype, B, w.q_heads, w.kv_heads, w.head_dim, w.page_size, seq_cap)
    for first in (None, torch.tensor([3, 0, 20], dtype=torch.int32, device="cuda")):
        out = gd.alloc(tuple(q.shape), q.dtype, fill=float("nan"))
        ctx.cast_tree_attention_rows(q, k, v, B, w.q_heads, w.kv_heads, w.head_dim, w.page_size, table, seq_cap, num_pages, kv,
                                     tr["anc"], tr["n_tree"], first, 0.0, out)
        assert ctx.cast_poll_status()[0] == 0
        ref = tree_attention(f32(q), f32(k), f32(v), w.page_size, tab, kv.cpu().numpy(), o["anc"], o["n_tree"])
        got = to_f64(out)
        for b in range(B):
            lo = int(first[b]) if first is not None else 0
            lo = min(lo, int(o["n_tree"][b]))
            assert np.isnan(got[b, :lo]).all() and np.isnan(got[b, int(o["n_tree"][b]):]).all()
            err = np.max(np.abs(got[b, lo: int(o["n_tree"][b])] - ref[b, lo: int(o["n_tree"][b])])) if lo < o["n_tree"][b] else 0.0
            assert err <= attention_tolerance(dtype)
    # acceptance, greedy and at temperature 1
    tl = wl.target_logits(w, "cpu")
    wl.plant_acceptance(w, tl, o["tokens"], o["parent"], o["n_tree"])
    tl = tl.cuda()
    alen, apath, bonus = gd.alloc((B,), torch.int32), gd.alloc((B, H + 1), torch.int32), gd.alloc((B,), torch.int32)
    ctx.cast_accept(tl, B, tr["tokens"], tr["parent"], tr["depth"], tr["anc"], tr["n_tree"], alen, apath, bonus)
    ol, op, ob = greedy_accept(to_f64(tl), o["tokens"], o["parent"], o["n_tree"], H)
    assert np.array_equal(alen.cpu().numpy(), ol) and np.array_equal(apath.cpu().numpy(), op)
    assert np.array_equal(bonus.cpu().numpy(), ob)
    s_tl, s_dl, ua, ub = wl.stochastic_accept_inputs(w, o["tokens"], o["parent"], o["n_tree"], "cuda", 0.7, Ncap)
    alen2, apath2, bonus2 = gd.alloc((B,), torch.int32), gd.alloc((B, H + 1), torch.int32), gd.alloc((B,), torch.int32)
    ctx.cast_accept_stochastic(s_tl, s_dl, B, 1.0, tr["tokens"], tr["parent"], tr["n_tree"], ua, ub, alen2, apath2, bonus2)
    assert ctx.cast_poll_status()[0] == 0
    from oracle import stochastic_accept
    sl, sp, sb, margin = stochastic_accept(to_f64(s_tl), to_f64(s_dl), o["tokens"], o["parent"], o["n_tree"], H, 1.0,
                                           ua.cpu().numpy(), ub.cpu().numpy())
    assert margin.min() >= 1e-9
    assert np.array_equal(alen2.cpu().numpy(), sl) and np.array_equal(apath2.cpu().numpy(), sp)
    assert np.array_equal(bonus2.cpu().numpy(), sb)
    torch.cuda.synchronize()
    gd.check()


# ------------------------------------------------------------------ run-to-run determinism
@pytest.mark.parametrize("name", ["c2_llama8b", "c3_llama8b_b16", "c4_llama70b_n64"])
def test_repeated_calls_give_identical_bits(binding, name):
    """No result depends on which CTA finishes first: the merges (cluster, ticket) combine their pieces in a
    fixed order, so a repeated call reproduces every output bit for bit - tree, attention (cluster mode,
    global-merge mode) and acceptance at temperature 1."""
    w = wl.CONFIGS[name]
    B, H = w.batch, w.depth
    kw = cfg_kwargs(w)
    ctx = binding.CastContext(max_batch=B, **kw)
    if w.cost_model:
        ctx.cast_set_cost_tables(B, *make_tables(w, B))
    root, kv = wl.root_tokens(w, "cpu").cuda(), wl.kv_lengths(w, "cpu").cuda()
    logits = [wl.draft_logits(w, l, "cuda") for l in range(1, H + 1)]
    q = wl.query(w, 0, "cuda")
    k, v = wl.kv_cache(w, 0, "cuda")
    table, num_pages = wl.page_table(w, "cuda")
    runs = []
    for rep in range(3):
        g = gpu_tree(ctx, root, kv, logits)
        d = g["dev"]
        out = gpu_attention(ctx, w, q, k, v, table, num_pages, kv, d["anc"], d["n_tree"])
        res = [g[key].tobytes() for key in ("tokens", "parent", "depth", "anc", "pool_idx", "scores", "n_tree")]
        res.append(out.view(torch.int16).cpu().numpy().tobytes())
        if rep == 0:
            sto = wl.stochastic_accept_inputs(w, g["tokens"], g["parent"], g["n_tree"], "cuda", 0.7)
        alen = torch.empty((B,), dtype=torch.int32, device="cuda")
        apath = torch.empty((B, H + 1), dtype=torch.int32, device="cuda")
        bonus = torch.empty((B,), dtype=torch.int32, device="cuda")
        ctx.cast_accept_stochastic(sto[0], sto[1], B, 1.0, d["tokens"], d["parent"], d["n_tree"], sto[2], sto[3], alen, apath, bonus)
        res += [alen.cpu().numpy().tobytes(), apath.cpu().numpy().tobytes(), bonus.cpu().numpy().tobytes()]
        assert ctx.cast_poll_status()[0] == 0
        runs.append(res)
    assert runs[0] == runs[1] == runs[2]


# ------------------------------------------------------------------ malformed inputs: a status, never a fault
def test_malformed_inputs_are_reported_not_followed(binding):
    """What the host can see is refused with a code; what only the device can see (a parent that does not
    precede its child, a tree larger than the budget, a path entry below zero) sets the status word, first
    error first, and the call still ends in bounds."""
    with pytest.raises(binding.CastError) as e:  # more children per node than the vocabulary has tokens
        binding.CastContext(max_batch=1, vocab=3, top_k=4, max_depth=2, total_token=8)
    assert e.value.code == 3
    with pytest.raises(binding.CastError) as e:  # token budget beyond the row stride
        binding.CastContext(max_batch=1, vocab=100, top_k=2, max_depth=2, total_token=64, max_tree=32)
    assert e.value.code == 3
    H, Ncap, V, B = 4, 32, 64, 2
    ctx = binding.CastContext(max_batch=B, vocab=V, top_k=2, max_depth=H, total_token=16, max_tree=Ncap)
    dev = lambda a: torch.from_numpy(a).cuda()
    tokens = np.zeros((B, Ncap), dtype=np.int32)
    parent = np.full((B, Ncap), -1, dtype=np.int32)
    parent[:, 1:6] = [0, 0, 1, 5, 2]  # node 4 names node 5 as its parent
    n_tree = np.array([6, 6], dtype=np.int32)
    logits = torch.zeros((B, Ncap, V), device="cuda")
    alen = torch.zeros(B, dtype=torch.int32, device="cuda")
    apath = torch.zeros((B, H + 1), dtype=torch.int32, device="cuda")
    bonus = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.cast_accept(logits, B, dev(tokens), dev(parent), None, None, dev(n_tree), alen, apath, bonus)
    st, detail = ctx.cast_poll_status()
    assert st == 6 and detail % Ncap == 4  # BAD_TREE, at the offending node
    assert int(alen.min()) >= 0 and int(alen.max()) <= H and ctx.cast_poll_status()[0] == 0
    # acceptance of a tree larger than the context's token budget: refused (its rows past the budget are not swept)
    parent_ok = np.full((B, Ncap), -1, dtype=np.int32)
    parent_ok[:, 1:20] = np.arange(0, 19)
    ctx.cast_accept(logits, B, dev(tokens), dev(parent_ok), None, None, dev(np.array([20, 6], dtype=np.int32)), alen, apath,
                    bonus)
    st, detail = ctx.cast_poll_status()
    assert st == 6 and detail == 0  # BAD_TREE, sequence 0
    assert int(alen[0]) == 0 and int(apath[0, 0]) == -1 and int(alen[1]) >= 0
    # attention with a tree larger than the context's token budget (tensor-core path)
    w = wl.Workload("bad", 700, B, "bf16", "f32", 8, 2, 128, 50, 60, 16, V, 1.0, H, 2, 16, False, 1, max_tree=Ncap)
    q = wl.query(w, 0, "cuda")
    k, v = wl.kv_cache(w, 0, "cuda")
    table, num_pages = wl.page_table(w, "cuda")
    kv = wl.kv_lengths(w, "cuda")
    anc = torch.zeros((B, Ncap, ctx.words), dtype=torch.int32, device="cuda")
    out = torch.zeros_like(q)
    ctx.cast_reserve_attention(q.dtype, B, 8, 2, 128, 16, wl.seq_capacity(w) // 16)
    ctx.cast_tree_attention(q, k, v, B, 8, 2, 128, 16, table, wl.seq_capacity(w) // 16, num_pages, kv, anc,
                            dev(np.array([20, 4], dtype=np.int32)), 0.0, out)
    assert ctx.cast_poll_status()[0] == 6
    # compaction with a path entry below zero inside the accepted length
    kk, vv = k.unsqueeze(0).contiguous(), v.unsqueeze(0).contiguous()
    path = np.full((B, H + 1), -1, dtype=np.int32)
    path[:, 0] = 0
    ctx.cast_compact_kv(kk, vv, B, 1, kk[0].numel() * 2, 2, 128, 16, table, wl.seq_capacity(w) // 16, num_pages, dev(path),
                        dev(np.array([2, 0], dtype=np.int32)), kv.clone())
    assert ctx.cast_poll_status()[0] == 7  # BAD_PAGE
    assert ctx.cast_poll_status()[0] == 0
    # a path that does not climb (entry j below j) next to the end of the sequence's capacity: the sources are
    # in range, the destinations would not be. Reported, nothing stored, the length left alone.
    cap = wl.seq_capacity(w)
    near_end = torch.tensor([cap - 1, cap - 1], dtype=torch.int32, device="cuda")
    path = np.zeros((B, H + 1), dtype=np.int32)  # 0, 0, 0
    k0, v0 = kk.clone(), vv.clone()
    lens = near_end.clone()
    ctx.cast_compact_kv(kk, vv, B, 1, kk[0].numel() * 2, 2, 128, 16, table, cap // 16, num_pages, dev(path),
                        dev(np.array([2, 2], dtype=np.int32)), lens)
    assert ctx.cast_poll_status()[0] == 7
    assert torch.equal(kk.view(torch.int16), k0.view(torch.int16)) and torch.equal(vv.view(torch.int16), v0.view(torch.int16))
    assert torch.equal(lens, near_end)
