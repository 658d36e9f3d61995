"""Randomised parity: many small configurations drawn from a fixed seed, each compared with the
oracle like the hand-picked cases of test_gpu_parity.py.  The draws cover what those cases fix by
hand: vocabulary sizes that are not multiples of anything, every K and W up to the caps, batch
sizes, logit dtypes, the sizing switches, window starts and head groupings."""
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
