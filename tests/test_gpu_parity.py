"""Parity of the CUDA library (through its C-ABI) with the CPU oracle on the same
seeded inputs.  Integer outputs (tree structure, indices, accept results,
compacted KV bytes) must be bit-exact; attention within max-abs 1e-5 (fp32
inputs) / 2e-2 (bf16 inputs)."""
import numpy as np
import pytest
import torch

from oracle import ancestor_masks, compact_kv, greedy_accept, stochastic_accept, tree_attention
from paper_2510_26577_b200 import workloads as wl

from helpers import (alloc_tree_outputs, assert_tree_equal, attention_tolerance, cfg_kwargs, gpu_attention, gpu_tree, make_tables,
                     oracle_tree, to_f64)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2510_26577_b200 import build
    build.build()
    from paper_2510_26577_b200 import binding as b
    b.load_library()
    return b


def _oracle_tables(w, B, stepped=False, skewed=False):
    from oracle import CostTable
    L, M, Ntab, fT, fD = make_tables(w, B, stepped, skewed)
    return {B: CostTable(B, L, M, Ntab, fT, fD)}, (L, M, Ntab, fT, fD)


def build_tree_both(binding, w, peaked=False, stepped=False, steps=1, skewed=False, **over):
    kw = cfg_kwargs(w, **over)
    B = w.batch
    need = kw.get("enable_bp") or kw.get("enable_dp") or kw.get("enable_dr")
    tables, raw = _oracle_tables(w, B, stepped, skewed) if need else (None, None)
    ctx = binding.CastContext(max_batch=B, **kw)
    if need:
        ctx.cast_set_cost_tables(B, *raw)
    root = wl.root_tokens(w, "cpu").cuda()
    kv = wl.kv_lengths(w, "cpu").cuda()
    oracle = None
    for step in range(steps):
        logits = [wl.draft_logits(w, 10 * step + l, "cpu", peaked=peaked, width=over.get("max_width", 0)).cuda()
                  for l in range(1, w.depth + 1)]
        o = oracle_tree(kw, tables, root, kv, logits, oracle)
        oracle = o["oracle"]
        g = gpu_tree(ctx, root, kv, logits)
        assert o["min_score_gap"] >= 1e-5 and o["stable"], \
            f"seed sits on a decision boundary (gap {o['min_score_gap']:.2e}, stable {o['stable']}): pick another seed"
        assert_tree_equal(g, o)
    return ctx, g, o, root, kv


def check_attention(binding, ctx, w, g, o, kv, layer=0, sample=None, dense=()):
    """sample: that many random (sequence, token, head) outputs; dense: (sequence, kv-head) pairs of which
    EVERY output is compared - all tree tokens times all heads of the group, i.e. every row of every 128-row
    block of that pair (the full ones and the ragged last one), every tile and every KV split it has."""
    q = wl.query(w, layer, "cpu").cuda()
    k, v = (t.cuda() for t in wl.kv_cache(w, layer, "cpu"))
    table, num_pages = wl.page_table(w, "cuda")
    out = gpu_attention(ctx, w, q, k, v, table, num_pages, kv, g["dev"]["anc"], g["dev"]["n_tree"])
    f32 = lambda t: t.float().cpu().numpy()
    tab = table.cpu().numpy() if table is not None else None
    B = w.batch
    only = None
    if sample is not None:
        rng = np.random.default_rng(5)
        only = set()
        for _ in range(sample):
            b = int(rng.integers(0, B))
            only.add((b, int(rng.integers(0, o["n_tree"][b])), int(rng.integers(0, w.q_heads))))
        for b in range(B):  # always include the last tree token (deepest mask) of head 0
            only.add((b, int(o["n_tree"][b]) - 1, 0))
        G = w.q_heads // w.kv_heads
        for b, kvh in dense:
            only |= {(b, t, h) for t in range(int(o["n_tree"][b])) for h in range(kvh * G, (kvh + 1) * G)}
    ref = tree_attention(f32(q), f32(k), f32(v), w.page_size, tab, kv.cpu().numpy(), o["anc"], o["n_tree"], None, only)
    got = to_f64(out)
    tol = attention_tolerance(w.kv_dtype)
    if only is None:
        for b in range(B):
            nb = int(o["n_tree"][b])
            assert np.isnan(got[b, nb:]).all() and np.isfinite(got[b, :nb]).all()
            got[b, nb:] = 0.0
        err = np.max(np.abs(got - ref))
    else:
        err = max(np.max(np.abs(got[b, t, h] - ref[b, t, h])) for (b, t, h) in only)
        for b in range(B):  # rows beyond the tree are left untouched (the helper pre-fills NaN)
            assert np.isnan(got[b, int(o["n_tree"][b]):]).all()
    print(f"{w.name}: attention max-abs error {err:.3e} over {'all' if only is None else len(only)} outputs")
    assert err <= tol, f"attention max-abs error {err:.3e} > {tol}"
    return err


def check_accept_and_compact(binding, ctx, w, g, o, kv):
    B, H = w.batch, w.depth
    tl = wl.target_logits(w, "cpu").cuda()
    wl.plant_acceptance(w, tl, o["tokens"], o["parent"], o["n_tree"])
    alen = torch.empty((B,), dtype=torch.int32, device="cuda")
    apath = torch.empty((B, H + 1), dtype=torch.int32, device="cuda")
    bonus = torch.empty((B,), dtype=torch.int32, device="cuda")
    d = g["dev"]
    ctx.cast_accept(tl, B, d["tokens"], d["parent"], d["depth"], d["anc"], d["n_tree"], alen, apath, bonus)
    nmax = int(o["n_tree"].max())
    ol, op, ob = greedy_accept(to_f64(tl[:, :nmax]), o["tokens"], o["parent"], o["n_tree"], H)
    assert ctx.cast_poll_status()[0] == 0
    assert np.array_equal(alen.cpu().numpy(), ol), (alen.cpu().numpy(), ol)
    assert np.array_equal(apath.cpu().numpy(), op)
    assert np.array_equal(bonus.cpu().numpy(), ob)
    # compaction over two layers of cache, compared as raw bytes
    k0, v0 = (t.cuda() for t in wl.kv_cache(w, 0, "cpu"))
    k1, v1 = (t.cuda() for t in wl.kv_cache(w, 1, "cpu"))
    kk, vv = torch.stack([k0, k1]).contiguous(), torch.stack([v0, v1]).contiguous()
    del k0, k1, v0, v1
    table, num_pages = wl.page_table(w, "cuda")
    bits = torch.int16 if w.kv_dtype == "bf16" else torch.int32
    k_old, v_old = kk.view(bits).cpu().numpy(), vv.view(bits).cpu().numpy()
    kv2 = kv.clone()
    ctx.cast_compact_kv(kk, vv, B, 2, kk[0].numel() * kk.element_size(), w.kv_heads, w.head_dim, w.page_size, table,
                        wl.seq_capacity(w) // (w.page_size or 1), num_pages, apath, alen, kv2)
    assert ctx.cast_poll_status()[0] == 0
    tab = table.cpu().numpy() if table is not None else None
    nk, nv, nlen = compact_kv(k_old, v_old, w.page_size, tab, kv.cpu().numpy(), op, ol)
    assert np.array_equal(kv2.cpu().numpy(), nlen)
    assert np.array_equal(kk.view(bits).cpu().numpy(), nk)
    assert np.array_equal(vv.view(bits).cpu().numpy(), nv)
    return ol


# ------------------------------------------------------------------ the five configurations
def test_c1_tiny_full_step(binding):
    w = wl.CONFIGS["c1_tiny"]
    ctx, g, o, root, kv = build_tree_both(binding, w)
    assert list(o["n_tree"]) == [16] and o["pool_size"] == 53
    check_attention(binding, ctx, w, g, o, kv)
    check_accept_and_compact(binding, ctx, w, g, o, kv)


def test_c2_llama8b_full_step(binding):
    w = wl.CONFIGS["c2_llama8b"]
    ctx, g, o, root, kv = build_tree_both(binding, w)
    assert list(o["n_tree"]) == [60] and o["pool_size"] == 511
    check_attention(binding, ctx, w, g, o, kv)
    ol = check_accept_and_compact(binding, ctx, w, g, o, kv)
    assert ol[0] >= 1  # planted acceptance gives the walk something to do
    # the same tree through the acceptance rule at temperature 1 and 0.6
    for T, salt in ((1.0, 0), (0.6, 1)):
        _run_stochastic(binding, ctx, wl.shrink(w, seed_salt=salt), o["tokens"], o["parent"], o["n_tree"], w.depth, T, 0.7)


@pytest.mark.parametrize("name", ["c3_llama8b_b1", "c3_llama8b_b4", "c3_llama8b_b16"])
def test_c3_batch_sweep_cost_model(binding, name):
    w = wl.CONFIGS[name]
    ctx, g, o, root, kv = build_tree_both(binding, w)
    assert 1 <= int(o["n_tree"][0]) <= 64
    # every output of the longest, the shortest and one more sequence for two kv-heads each (global-merge
    # launch at batch 16: all splits and the merge of those pairs), and of every (sequence, kv-head) pair below
    lens = kv.cpu().numpy()
    seqs = sorted({int(np.argmax(lens)), int(np.argmin(lens)), w.batch // 2})
    dense = [(b, h) for b in seqs for h in (0, w.kv_heads - 1)] if w.batch > 1 else [(0, h) for h in range(w.kv_heads)]
    check_attention(binding, ctx, w, g, o, kv, sample=24, dense=dense)
    check_accept_and_compact(binding, ctx, w, g, o, kv)
    if name == "c3_llama8b_b16":  # more sequences than clusters fit at a time
        _run_stochastic(binding, ctx, w, o["tokens"], o["parent"], o["n_tree"], w.depth, 1.0, 0.7)


@pytest.mark.parametrize("name", ["c3_llama8b_b4", "c3_llama8b_b16"])
def test_c3_rerank_per_sequence_ragged_trees(binding, name):
    # every sequence sizes its own tree in the rerank: n_tree differs per sequence, and the attention,
    # acceptance and compaction that follow work on ragged trees
    # (batch 4: the default seed puts one sequence's rerank within rounding of its threshold; the oracle's
    # stability flag says so, and the recipe's answer to that is another seed)
    w = wl.shrink(wl.CONFIGS[name], seed_salt=2 if name == "c3_llama8b_b4" else 0)
    ctx, g, o, root, kv = build_tree_both(binding, w, rerank_per_row=1)
    sizes = [int(x) for x in o["n_tree"]]
    assert len(set(sizes)) > 1 and 1 <= min(sizes) and max(sizes) <= 64, sizes
    check_attention(binding, ctx, w, g, o, kv, sample=24)
    check_accept_and_compact(binding, ctx, w, g, o, kv)
    if name == "c3_llama8b_b4":
        _run_stochastic(binding, ctx, w, o["tokens"], o["parent"], o["n_tree"], w.depth, 1.0, 0.7)


def test_c3_b64_tree_and_accept_reduced_vocab(binding):
    # batch 64 with the full 128k vocabulary takes the oracle minutes; the vocabulary is cut to 8k here
    # (the full-size launch is exercised by bench.py and checked there against invariants)
    w = wl.shrink(wl.CONFIGS["c3_llama8b_b64"], vocab=8192, kv_len_lo=64, kv_len_hi=300, seed_salt=1)
    ctx, g, o, root, kv = build_tree_both(binding, w)
    check_attention(binding, ctx, w, g, o, kv, sample=32)
    check_accept_and_compact(binding, ctx, w, g, o, kv)


def test_c3_b64_full_vocab_tree_accept_compaction(binding):
    # batch 64 at the full 128k vocabulary: tree build (the oracle needs half a minute for its 3000 row sorts), then
    # acceptance and compaction on that tree
    w = wl.CONFIGS["c3_llama8b_b64"]
    ctx, g, o, root, kv = build_tree_both(binding, w)
    assert 4 <= int(o["n_tree"][0]) <= 16  # the cost model shrinks the tree at batch 64
    # acceptance (argmax sweep over 64 x N rows of the full vocabulary) and compaction at the same size
    check_accept_and_compact(binding, ctx, w, g, o, kv)


@pytest.mark.parametrize("name", ["c4_llama70b_n16", "c4_llama70b_n32", "c4_llama70b_n128"])
def test_c4_llama70b(binding, name):
    w = wl.CONFIGS[name]
    ctx, g, o, root, kv = build_tree_both(binding, w)
    assert list(o["n_tree"]) == [w.total_token] * 8
    # every output of two (sequence, kv-head) pairs: with 128 tokens x 8 heads that is eight full 128-row
    # blocks each, the tree spanning two 64-position tiles, and every KV split of the global-merge launch
    check_attention(binding, ctx, w, g, o, kv, sample=16, dense=[(0, 0), (5, 7)])
    check_accept_and_compact(binding, ctx, w, g, o, kv)
    _run_stochastic(binding, ctx, w, o["tokens"], o["parent"], o["n_tree"], w.depth, 1.0, 0.7)


def test_c5_qwen_long_context(binding):
    w = wl.CONFIGS["c5_qwen_long"]
    ctx, g, o, root, kv = build_tree_both(binding, w)
    assert list(o["n_tree"]) == [96] * 4
    # every output of one (sequence, kv-head) pair: 96 tokens x 7 heads = five full 128-row blocks and a
    # ragged one of 32 rows, 515 tiles in 8 splits each
    check_attention(binding, ctx, w, g, o, kv, sample=8, dense=[(1, 2)])
    check_accept_and_compact(binding, ctx, w, g, o, kv)
    _run_stochastic(binding, ctx, w, o["tokens"], o["parent"], o["n_tree"], w.depth, 0.9, 0.5)  # the largest cached slice


# ------------------------------------------------------------------ tree-build variants and edge cases
SMALL = wl.Workload("small", 77, 3, "f32", "f32", 4, 2, 64, 5, 40, 0, 1001, 2.0, 4, 3, 20, False, 2, max_tree=32)


def test_unaligned_vocab_and_bf16_ties(binding):
    # V = 1001 breaks 16-byte row alignment; bf16 logits tie often, so the token-id tie-break is exercised
    build_tree_both(binding, SMALL)
    build_tree_both(binding, wl.shrink(SMALL, logit_dtype="bf16", config_id=78, vocab=5000, logit_std=0.05))


@pytest.mark.parametrize("over", [
    dict(vocab=3000, top_k=16, depth=2, batch=2, total_token=64, max_tree=64, config_id=81),  # K = W = 16: the caps
    dict(vocab=20, top_k=3, depth=3, batch=1, total_token=10, config_id=82),      # fewer logits than lanes
    dict(vocab=70001, top_k=8, depth=2, batch=2, logit_dtype="bf16", logit_std=3.0, config_id=83),  # 8 ragged chunks
    dict(vocab=200000, top_k=5, depth=2, batch=1, logit_std=3.0, config_id=84),   # chunks of more than one pass
])
def test_tree_build_shapes(binding, over):
    build_tree_both(binding, wl.shrink(SMALL, **over))


def test_uniform_and_neg_inf_logits(binding):
    w = wl.shrink(SMALL, batch=1, vocab=4096, config_id=79)
    kw = cfg_kwargs(w)
    ctx = binding.CastContext(max_batch=1, **kw)
    root, kv = wl.root_tokens(w, "cpu").cuda(), wl.kv_lengths(w, "cpu").cuda()
    logits = [torch.zeros((1, 3, 4096), device="cuda") for _ in range(w.depth)]
    for lg in logits:
        lg[:, :, 100:] = float("-inf")  # probability 0 outside the first 100 tokens
    o = oracle_tree(kw, None, root, kv, logits)
    g = gpu_tree(ctx, root, kv, logits)
    assert_tree_equal(g, o)
    assert np.allclose(o["scores"][0, 1:4], -np.log(100), atol=1e-12)  # closed form


def test_nan_logits_raise_device_status(binding):
    w = wl.shrink(SMALL, batch=1, config_id=80)
    ctx = binding.CastContext(max_batch=1, **cfg_kwargs(w))
    root, kv = wl.root_tokens(w, "cpu").cuda(), wl.kv_lengths(w, "cpu").cuda()
    logits = [wl.draft_logits(w, l, "cpu").cuda() for l in range(1, w.depth + 1)]
    logits[1][0, 1, 17] = float("nan")
    g = gpu_tree(ctx, root, kv, logits)
    assert g["status"][0] == 8  # CAST_ERR_NONFINITE
    assert ctx.cast_poll_status()[0] == 0  # cleared by the poll


@pytest.mark.parametrize("over", [
    dict(enable_bp=1, enable_dr=1, C1=0.5, C3=0.3),
    dict(enable_bp=1, enable_dp=1, enable_dr=1, C1=0.3, C2=0.02, C3=0.2),
    dict(pool_mode=1),
    dict(enable_bp=1, enable_dr=1, ctx_base_mode=1, max_width=6, C1=0.2, C3=0.2),
])
def test_cost_model_switches_multi_step(binding, over):
    # peaked logits: values decay slowly, so breadth/depth pruning and the FIFO state all act; 3 steps
    w = wl.Workload("sw", 81, 4, "f32", "f32", 4, 2, 64, 100, 900, 0, 3000, 2.0, 5, 4, 24, False, 2, max_tree=32,
                    tau=4e-2)
    build_tree_both(binding, w, peaked=True, steps=3, **over)
    build_tree_both(binding, w, peaked=True, stepped=True, steps=2, **over)


@pytest.mark.parametrize("over", [
    dict(enable_bp=1, enable_dp=1, enable_dr=1, C1=0.6, C2=0.05, C3=0.25),
    dict(enable_bp=1, enable_dp=1, enable_dr=1, C1=0.25, C2=0.02, C3=0.6, max_width=6),
    dict(enable_bp=1, enable_dr=1, ctx_base_mode=1, C1=0.4, C3=0.15),
    dict(enable_dr=1, rerank_per_row=1, C3=0.3),
])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_cost_model_tables_where_a_wrong_lookup_shows(binding, over, seed):
    """Tables whose rows differ by tens of percent on a grid of 8 positions, f_D not a multiple of
    f_T, ragged prefixes that land in different rows, C1 != C3: a lookup in the wrong table, row
    or column, or a swapped threshold, changes the tree.  Three steps, so the depth-pruning
    buffers carry over.  A draw that sits within rounding of a threshold is skipped by the
    oracle's margin, not reseeded."""
    w = wl.Workload("skew", 83, 3, "f32", "f32", 4, 2, 64, 5, 300, 0, 2500, 2.0, 5, 4, 24, False, 2, max_tree=32,
                    tau=2.5e-2, seed_salt=seed)
    try:
        ctx, g, o, root, kv = build_tree_both(binding, w, peaked=True, steps=3, skewed=True, **over)
    except AssertionError as e:
        if "decision boundary" in str(e):
            pytest.skip(str(e))
        raise
    # the case must exercise the switches: some layer narrowed or stopped, and a rerank below the budget
    assert min(o["n_hist"]) < (over.get("max_width") or w.top_k) or len(o["n_hist"]) < w.depth or \
        int(o["n_tree"].min()) < w.total_token


def _golden_gpu_case(binding, case):
    kw = case.config_kwargs()
    B = case.B
    ctx = binding.CastContext(max_batch=B, **kw)
    if case.fT:
        ctx.cast_set_cost_tables(B, *case.table_arrays())
    root = torch.tensor(case.root, dtype=torch.int32, device="cuda")
    kv = torch.tensor(case.kv_len, dtype=torch.int32, device="cuda")
    H = int(case.param["H"])
    logits = [torch.from_numpy(case.logits(l)).float().cuda() for l in range(1, H + 1)]
    for step in case.steps():
        g = gpu_tree(ctx, root, kv, logits)
        assert g["status"][0] == 0
        layers = case.layers(step)
        assert g["info"]["layers"] == len(layers)
        for layer in layers:
            key = ("step", step, "layer", layer)
            n_i = case.ints(*key, "n")[0][0]
            nt, npr, cnt = g["per_layer"][layer - 1]
            assert g["info"]["n_hist"][layer - 1] == n_i, (key, g["info"]["n_hist"])
            assert cnt == case.ints(*key, "next_count")[0][0], key
            for b in range(B):
                assert list(nt[b, :n_i]) == case.ints(*key, "next_tokens")[b], (key, b)
                assert list(npr[b, :n_i]) == case.ints(*key, "next_parent_row")[b], (key, b)
        N = case.ints("step", step, "N")[0][0]
        assert list(g["n_tree"]) == [N] * B
        for name in ("tokens", "parent", "depth", "pool_idx"):
            for b in range(B):
                assert list(g[name][b, :N]) == case.ints("step", step, name)[b], (step, name, b)
        for b in range(B):
            assert list(g["anc"][b, :N, 0]) == case.ints("step", step, "anc")[b]
    return ctx


def test_hand_worked_step_on_the_gpu(binding):
    """The batch-2, two-step case derived by hand in tests/golden/cast_step_b2.txt (every sizing
    switch on; cost rows, tables and thresholds chosen so that a wrong lookup changes a decision)
    through the C-ABI: the library's decisions and trees against the hand-derived ones, not
    against the oracle."""
    import golden_cases

    (case,) = golden_cases.load("cast_step_b2.txt")
    ctx = _golden_gpu_case(binding, case)
    # the depth-pruning buffers after the two steps, read back through the state export
    import struct
    blob = ctx.cast_state_export()
    nbuf, R = struct.unpack_from("ii", blob, 0)
    off = 8
    for i, want in enumerate(case.get("step", 2, "fifo")):
        cnt, = struct.unpack_from("i", blob, off)
        vals = struct.unpack_from(f"{R}d", blob, off + 4)
        off += 4 + 8 * R
        assert cnt == len(want) and np.allclose(vals[:cnt], [float(v) for v in want], rtol=1e-6), (i, vals)


def test_state_export_import_roundtrip(binding):
    w = wl.Workload("st", 82, 2, "f32", "f32", 4, 2, 64, 100, 900, 0, 2000, 2.0, 4, 3, 16, False, 2, max_tree=32,
                    tau=4e-2)
    over = dict(enable_bp=1, enable_dp=1, enable_dr=1, C1=0.3, C2=0.02, C3=0.2, fifo_len=2)
    ctx, g, o, root, kv = build_tree_both(binding, w, peaked=True, steps=3, **over)
    blob = ctx.cast_state_export()
    fifo = o["oracle"].fifo
    import struct
    nbuf, R = struct.unpack_from("ii", blob, 0)
    assert (nbuf, R) == (w.depth - 1, 2)
    off = 8
    for i in range(nbuf):
        cnt, = struct.unpack_from("i", blob, off)
        vals = struct.unpack_from(f"{R}d", blob, off + 4)
        off += 4 + 8 * R
        assert cnt == len(fifo[i]) and np.allclose(vals[:cnt], fifo[i], rtol=1e-6)
    ctx2 = binding.CastContext(max_batch=w.batch, **cfg_kwargs(w, **over))
    ctx2.cast_state_import(blob)
    assert ctx2.cast_state_export() == blob


def test_host_side_argument_checks(binding):
    with pytest.raises(binding.CastError) as e:
        binding.CastContext(max_batch=1, vocab=100, top_k=17, max_depth=2, total_token=8)
    assert e.value.code == 3
    ctx = binding.CastContext(max_batch=2, vocab=100, top_k=2, max_depth=2, total_token=8, enable_bp=1)
    root = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.CastError) as e:  # a switch is on, no table for B=2
        ctx.cast_step_begin(2, root, root)
    assert e.value.code == 5
    with pytest.raises(binding.CastError) as e:  # cost not strictly increasing
        ctx.cast_set_cost_tables(2, 8, 1, 3, [1.0, 1.0, 2.0], [1.0, 2.0, 3.0])
    assert e.value.code == 5
    ctx.cast_set_cost_tables(2, 8, 1, 3, [1.0, 2.0, 3.0], [1.0, 2.0, 3.0])
    ctx.cast_step_begin(2, root, root)
    lg = torch.zeros((2, 2, 100), device="cuda")
    o = [torch.empty((2, 2), dtype=torch.int32, device="cuda") for _ in range(2)] + \
        [torch.empty(1, dtype=torch.int32, device="cuda")]
    with pytest.raises(binding.CastError) as e:  # layer 2 before layer 1
        ctx.cast_tree_expand(2, lg, *o)
    assert e.value.code == 1


# ------------------------------------------------------------------ attention on arbitrary trees
def _random_tree(rng, N, kind):
    if kind == "chain":
        parent = np.arange(-1, N - 1)
    elif kind == "star":
        parent = np.array([-1] + [0] * (N - 1))
    else:
        parent = np.array([-1] + [int(rng.integers(0, t)) for t in range(1, N)])
    return parent


@pytest.mark.parametrize("dtype,D,Hq,Hkv,page", [("f32", 64, 8, 8, 0), ("f32", 128, 8, 2, 16), ("bf16", 128, 32, 8, 16),
                                                 ("bf16", 128, 64, 8, 0), ("bf16", 64, 4, 4, 16),
                                                 ("bf16", 128, 28, 4, 16)])
def test_attention_arbitrary_trees_ragged(binding, dtype, D, Hq, Hkv, page):
    rng = np.random.default_rng(99)
    B, Ncap = 5, 128
    w = wl.Workload("attn", 90, B, dtype, "f32", Hq, Hkv, D, 0, 700, page, 100, 1.0, 4, 2, 8, False, 1)
    ctx = binding.CastContext(max_batch=B, vocab=100, top_k=2, max_depth=8, total_token=128, max_tree=Ncap)
    kv = torch.tensor([0, 1, 63, 700, 257], dtype=torch.int32, device="cuda")
    n_tree = np.array([1, 128, 37, 64, 5], dtype=np.int32)
    kinds = ["chain", "random", "star", "random", "chain"]
    anc = np.zeros((B, Ncap, 4), dtype=np.uint32)
    for b in range(B):
        anc[b] = np.pad(ancestor_masks(_random_tree(rng, int(n_tree[b]), kinds[b]), int(n_tree[b]), 4),
                        ((0, Ncap - int(n_tree[b])), (0, 0)))
    q = wl.query(w, 0, "cpu").cuda()
    k, v = (t.cuda() for t in wl.kv_cache(w, 0, "cpu"))
    table, num_pages = wl.page_table(w, "cuda")
    nt = torch.from_numpy(n_tree).cuda()
    # cache rows past a sequence's last tree token may hold anything: poison them with NaN
    cap = wl.seq_capacity(w)
    for b in range(B):
        end = int(kv[b]) + int(n_tree[b])
        if page:
            for pos in range(end, cap):
                pg = int(table[b, pos // page])
                k[pg, pos % page] = float("nan")
                v[pg, pos % page] = float("nan")
        else:
            k[b, end:] = float("nan")
            v[b, end:] = float("nan")
    # so may the query rows of tokens past the tree (they share 128-row blocks with live rows): NaN, inf, huge
    for b in range(B):
        nb = int(n_tree[b])
        q[b, nb::3] = float("nan")
        q[b, nb + 1::3] = float("inf")
        q[b, nb + 2::3] = 3.0e38
    out = gpu_attention(ctx, w, q, k, v, table, num_pages, kv, anc, nt, scale=0.0)
    assert ctx.cast_poll_status()[0] == 0
    f32 = lambda t: t.float().cpu().numpy()
    tab = table.cpu().numpy() if table is not None else None
    only = {(b, int(t), int(h)) for b in range(B) for t in rng.integers(0, n_tree[b], size=6)
            for h in rng.integers(0, Hq, size=3)}
    only |= {(b, int(n_tree[b]) - 1, Hq - 1) for b in range(B)}
    ref = tree_attention(f32(q), f32(k), f32(v), page, tab, kv.cpu().numpy(), anc, n_tree, None, only)
    got = to_f64(out)
    err = max(np.max(np.abs(got[i] - ref[i])) for i in only)
    assert err <= attention_tolerance(dtype), err
    for b in range(B):
        assert np.isnan(got[b, int(n_tree[b]):]).all()


@pytest.mark.parametrize("name", ["c1_tiny", "c2_llama8b", "c4_llama70b_n128"])
def test_attention_rows_of_the_growing_tree(binding, name):
    """The draft-side use: layer by layer, the new layer's tokens attend to the prefix and the earlier
    layers (the linear order is creation order, so the tree after layer d is a prefix of the final tree).
    c1: CUDA-core path; c2, c4: tensor-core path, cluster and global-merge launches."""
    w = wl.CONFIGS[name]
    ctx, g, o, root, kv = build_tree_both(binding, w)
    B, Hq = w.batch, w.q_heads
    q = wl.query(w, 0, "cpu").cuda()
    k, v = (t.cuda() for t in wl.kv_cache(w, 0, "cpu"))
    table, num_pages = wl.page_table(w, "cuda")
    tab = table.cpu().numpy() if table is not None else None
    f32 = lambda t: t.float().cpu().numpy()
    qf, kf, vf = f32(q), f32(k), f32(v)
    depth = o["depth"]
    assert all(np.all(np.diff(depth[b, : int(o["n_tree"][b])]) >= 0) for b in range(B))  # creation order is layer order
    rng = np.random.default_rng(3)
    for d in range(1, int(depth.max()) + 1):
        first = np.array([int(np.sum(depth[b, : int(o["n_tree"][b])] < d)) for b in range(B)], dtype=np.int32)
        end = np.array([int(np.sum(depth[b, : int(o["n_tree"][b])] <= d)) for b in range(B)], dtype=np.int32)
        out = gpu_attention(ctx, w, q, k, v, table, num_pages, kv, g["dev"]["anc"], torch.from_numpy(end).cuda(),
                            first_row=torch.from_numpy(first).cuda())
        assert ctx.cast_poll_status()[0] == 0
        got = to_f64(out)
        only = set()
        for b in range(B):
            assert np.isnan(got[b, : first[b]]).all() and np.isnan(got[b, end[b]:]).all()  # rows outside the window: untouched
            assert np.isfinite(got[b, first[b]: end[b]]).all()
            if first[b] == end[b]:  # this sequence kept nothing of layer d
                continue
            for t in {int(first[b]), int(end[b]) - 1} | {int(x) for x in rng.integers(first[b], end[b], size=2)}:
                for h in {0, Hq - 1, int(rng.integers(0, Hq))}:
                    only.add((b, t, h))
        ref = tree_attention(qf, kf, vf, w.page_size, tab, kv.cpu().numpy(), o["anc"], end, None, only)
        err = max(np.max(np.abs(got[i] - ref[i])) for i in only)
        assert err <= attention_tolerance(w.kv_dtype), (d, err)
    # an empty window writes nothing; a null first_row is the plain call
    nt = g["dev"]["n_tree"]
    out = gpu_attention(ctx, w, q, k, v, table, num_pages, kv, g["dev"]["anc"], nt, first_row=nt.clone())
    assert torch.isnan(out).all()


@pytest.mark.parametrize("name,n", [("c3_llama8b_b64", 9), ("c3_llama8b_b16", 12), ("c4_llama70b_n32", 32)])
def test_attention_full_size_launch_sampled(binding, name, n):
    """The launch shapes bench.py times (plain, global-merge and cluster mode at full cache sizes), on
    random trees of the size the tree build produces there; the oracle computes sampled outputs."""
    rng = np.random.default_rng(7)
    w = wl.CONFIGS[name]
    B, Ncap = w.batch, w.max_tree
    ctx = binding.CastContext(max_batch=B, **cfg_kwargs(w, enable_bp=0, enable_dr=0))
    kv = wl.kv_lengths(w, "cpu").cuda()
    n_tree = np.full(B, n, dtype=np.int32)
    anc = np.zeros((B, Ncap, 4), dtype=np.uint32)
    for b in range(B):
        anc[b, :n] = ancestor_masks(_random_tree(rng, n, "random"), n, 4)
    q = wl.query(w, 0, "cpu").cuda()
    k, v = (t.cuda() for t in wl.kv_cache(w, 0, "cpu"))
    table, num_pages = wl.page_table(w, "cuda")
    out = gpu_attention(ctx, w, q, k, v, table, num_pages, kv, anc, torch.from_numpy(n_tree).cuda(), scale=0.0)
    assert ctx.cast_poll_status()[0] == 0
    only = {(int(b), int(rng.integers(0, n)), int(rng.integers(0, w.q_heads))) for b in rng.integers(0, B, size=24)}
    only |= {(b, n - 1, w.q_heads - 1) for b in (0, B - 1)}
    # and every output (all tokens, all heads of the group) of the longest, the shortest and one more sequence
    # for the first and the last kv-head: every row block, tile and split of those pairs
    lens, G = kv.cpu().numpy(), w.q_heads // w.kv_heads
    for b in sorted({int(np.argmax(lens)), int(np.argmin(lens)), B // 2}):
        for kvh in (0, w.kv_heads - 1):
            only |= {(b, t, h) for t in range(n) for h in range(kvh * G, (kvh + 1) * G)}
    f32 = lambda t: t.float().cpu().numpy()
    tab = table.cpu().numpy() if table is not None else None
    ref = tree_attention(f32(q), f32(k), f32(v), w.page_size, tab, kv.cpu().numpy(), anc, n_tree, None, only)
    got = to_f64(out)
    err = max(np.max(np.abs(got[i] - ref[i])) for i in only)
    print(f"{name}: attention max-abs error {err:.3e} over {len(only)} outputs")
    assert err <= attention_tolerance(w.kv_dtype), err
    for b in (0, B - 1):
        assert np.isnan(got[b, n:]).all()


@pytest.mark.parametrize("name,factor", [("c2_llama8b", 12.0), ("c4_llama70b_n128", 12.0), ("c3_llama8b_b64", 12.0),
                                         ("c2_llama8b", 60.0)])
def test_attention_score_far_above_the_earlier_tiles(binding, name, factor):
    """A key far better than anything before it, met late: in the last prefix tile, in a tree tile and in
    the middle of the prefix (the scores of the tiles before it are ordinary, so the running reference of
    the single-pass softmax is ~100 to ~700 nats too low when the key arrives). Cluster, global-merge and
    plain launches; compared with the oracle on the planted rows and on their neighbours."""
    rng = np.random.default_rng(11)
    w = wl.CONFIGS[name]
    B, Ncap, Hq, G = w.batch, w.max_tree, w.q_heads, w.q_heads // w.kv_heads
    n = min(w.total_token, 16) if name.startswith("c3") else w.total_token
    ctx = binding.CastContext(max_batch=B, **cfg_kwargs(w, enable_bp=0, enable_dr=0))
    kv = wl.kv_lengths(w, "cpu").cuda()
    kvh_ = kv.cpu().numpy()
    n_tree = np.full(B, n, dtype=np.int32)
    anc = np.zeros((B, Ncap, 4), dtype=np.uint32)
    for b in range(B):
        anc[b, :n] = ancestor_masks(_random_tree(rng, n, "random"), n, 4)
    q = wl.query(w, 0, "cpu")
    k, v = wl.kv_cache(w, 0, "cpu")
    table, num_pages = wl.page_table(w, "cpu")
    only = set()

    def plant(b, t, h, pos):
        row = (q[b, t, h].float() * factor).to(k.dtype)
        if w.page_size:
            k[int(table[b, pos // w.page_size]), pos % w.page_size, h // G] = row
        else:
            k[b, pos, h // G] = row
        for tt in {t, max(t - 1, 0), min(t + 1, n - 1)}:
            for hh in range(h // G * G, h // G * G + G):
                only.add((b, tt, hh))

    bs = sorted({0, B - 1, B // 2})
    for i, b in enumerate(bs):
        L = int(kvh_[b])
        t = n - 1 - i  # a late tree token: its own tree position is in the last tile
        plant(b, t, (3 * i) % Hq, L - 1 - 5 * i)          # last prefix tile
        plant(b, t, (G + 1 + 3 * i) % Hq, L + t)          # its own position in the tree (always visible)
        plant(b, 1 + i, (2 * G + 2 + i) % Hq, L // 2 + 7)  # middle of the prefix: a later split's first tiles
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    td = table.cuda() if table is not None else None
    out = gpu_attention(ctx, w, qd, kd, vd, td, num_pages, kv, anc, torch.from_numpy(n_tree).cuda(), scale=0.0)
    assert ctx.cast_poll_status()[0] == 0
    f32 = lambda t_: t_.float().numpy()
    tab = table.numpy() if table is not None else None
    if len(only) > 400:
        keep = sorted(only)
        only = {keep[i] for i in rng.permutation(len(keep))[:400]}
    ref = tree_attention(f32(q), f32(k), f32(v), w.page_size, tab, kvh_, anc, n_tree, None, only)
    got = to_f64(out)
    assert np.isfinite(got[:, :n]).all()
    err = max(np.max(np.abs(got[i] - ref[i])) for i in only)
    assert err <= attention_tolerance(w.kv_dtype), err


@pytest.mark.parametrize("name", ["c2_llama8b", "c3_llama8b_b16", "c4_llama70b_n32"])
@pytest.mark.parametrize("shift", [-3000.0, -700.0, 900.0, "mixed"])
def test_attention_all_scores_far_from_zero(binding, name, shift):
    """Every score of a head lies hundreds of nats below (or above) zero: the softmax's reference starts at 0
    and has to move down (everything would underflow) or up (everything would overflow) in the first tile of
    every piece. The keys get a component along the head's mean query, which shifts all its scores; "mixed"
    gives the kv-heads different shifts and leaves some untouched, so that one launch has rows that move up,
    rows that move down and rows that stay. Cluster and global-merge launches; sampled outputs vs the oracle."""
    rng = np.random.default_rng(23)
    w = wl.CONFIGS[name]
    B, Ncap, Hq, Hkv = w.batch, w.max_tree, w.q_heads, w.kv_heads
    G = Hq // Hkv
    n = 12 if name.startswith("c3") else w.total_token
    ctx = binding.CastContext(max_batch=B, **cfg_kwargs(w, enable_bp=0, enable_dr=0))
    kv = wl.kv_lengths(w, "cpu").cuda()
    kvh_ = kv.cpu().numpy()
    n_tree = np.full(B, n, dtype=np.int32)
    anc = np.zeros((B, Ncap, 4), dtype=np.uint32)
    for b in range(B):
        anc[b, :n] = ancestor_masks(_random_tree(rng, n, "random"), n, 4)
    q = wl.query(w, 0, "cpu")
    k, v = wl.kv_cache(w, 0, "cpu")
    table, num_pages = wl.page_table(w, "cpu")
    # all queries of a kv-head's group point roughly the same way (u plus noise), the keys get c * u added:
    # every score of the group moves by about c * |u|^2 = the wanted shift in raw score units
    scale = 1.0 / np.sqrt(w.head_dim)
    for kvh in range(Hkv):
        sh = shift if shift != "mixed" else [-3000.0, 0.0, 900.0, -200.0][kvh % 4]
        if sh == 0.0:
            continue
        u = torch.randn(w.head_dim, generator=torch.Generator().manual_seed(100 + kvh))
        u = u / u.norm() * 4.0
        q[:, :, kvh * G:(kvh + 1) * G] = (u + 0.3 * q[:, :, kvh * G:(kvh + 1) * G].float()).to(q.dtype)
        c = (sh / scale) / float(u.norm() ** 2)  # nats -> raw score units
        if w.page_size:
            k[:, :, kvh] = (k[:, :, kvh].float() + c * u).to(k.dtype)
        else:
            k[:, :, kvh] = (k[:, :, kvh].float() + c * u).to(k.dtype)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    td = table.cuda() if table is not None else None
    out = gpu_attention(ctx, w, qd, kd, vd, td, num_pages, kv, anc, torch.from_numpy(n_tree).cuda(), scale=0.0)
    assert ctx.cast_poll_status()[0] == 0
    only = {(int(rng.integers(0, B)), int(rng.integers(0, n)), int(rng.integers(0, Hq))) for _ in range(40)}
    only |= {(b, n - 1, h) for b in (0, B - 1) for h in range(0, Hq, max(1, G))}
    f32 = lambda t_: t_.float().numpy()
    tab = table.numpy() if table is not None else None
    ref = tree_attention(f32(q), f32(k), f32(v), w.page_size, tab, kvh_, anc, n_tree, None, only)
    got = to_f64(out)
    assert np.isfinite(got[:, :n]).all()
    err = max(np.max(np.abs(got[i] - ref[i])) for i in only)
    assert err <= attention_tolerance(w.kv_dtype), err


def test_attention_bad_page_sets_status(binding):
    w = wl.Workload("attnbad", 91, 1, "bf16", "f32", 8, 2, 128, 100, 100, 16, 100, 1.0, 4, 2, 8, False, 1)
    ctx = binding.CastContext(max_batch=1, vocab=100, top_k=2, max_depth=4, total_token=8)
    q = wl.query(w, 0, "cpu").cuda()
    k, v = (t.cuda() for t in wl.kv_cache(w, 0, "cpu"))
    table, num_pages = wl.page_table(w, "cuda")
    table[0, 2] = num_pages + 5
    anc = np.zeros((1, 128, 4), dtype=np.uint32)
    anc[0, :4] = ancestor_masks(np.array([-1, 0, 1, 2]), 4, 4)
    gpu_attention(ctx, w, q, k, v, table, num_pages, wl.kv_lengths(w, "cpu").cuda(), anc,
                  torch.tensor([4], dtype=torch.int32, device="cuda"))
    assert ctx.cast_poll_status()[0] == 7


# ------------------------------------------------------------------ accept / compaction edge cases
def test_accept_edge_cases_and_overlapping_compaction(binding):
    H = 4
    ctx = binding.CastContext(max_batch=3, vocab=64, top_k=2, max_depth=H, total_token=8, max_tree=32)
    Ncap, V = 32, 64
    tokens = np.full((3, Ncap), -1, dtype=np.int32)
    parent = np.full((3, Ncap), -1, dtype=np.int32)
    tokens[:, :5] = [7, 3, 4, 5, 6]
    parent[:, :5] = [-1, 0, 0, 2, 3]
    n_tree = np.array([5, 5, 3], dtype=np.int32)
    logits = torch.zeros((3, Ncap, V), device="cuda")
    # row 0: nothing matches (all-zero logits: argmax 0). rows 1, 2: 0 -> 2 -> 3 -> 4
    for b in (1, 2):
        logits[b, 0, 4] = 1; logits[b, 2, 5] = 1; logits[b, 3, 6] = 1; logits[b, 4, 9] = 1
    dev = lambda a: torch.from_numpy(a).cuda()
    alen = torch.empty(3, dtype=torch.int32, device="cuda")
    apath = torch.empty((3, H + 1), dtype=torch.int32, device="cuda")
    bonus = torch.empty(3, dtype=torch.int32, device="cuda")
    ctx.cast_accept(logits, 3, dev(tokens), dev(parent), None, None, dev(n_tree), alen, apath, bonus)
    ol, op, ob = greedy_accept(to_f64(logits), tokens, parent, n_tree, H)
    assert list(ol) == [0, 3, 1]
    assert np.array_equal(alen.cpu().numpy(), ol) and np.array_equal(apath.cpu().numpy(), op)
    assert np.array_equal(bonus.cpu().numpy(), ob)
    # compaction with an overlapping path (0,2,3,4): slot 2 is a destination and a later source
    for page in (0, 4):
        w = wl.Workload("cmp", 92, 3, "f32", "f32", 2, 2, 64, 3, 9, page, 64, 1.0, H, 2, 8, False, 3, max_tree=32)
        kv = wl.kv_lengths(w, "cpu").cuda()
        layers = [tuple(t.cuda() for t in wl.kv_cache(w, l, "cpu")) for l in range(3)]
        kk = torch.stack([a for a, _ in layers]).contiguous()
        vv = torch.stack([b for _, b in layers]).contiguous()
        table, num_pages = wl.page_table(w, "cuda")
        k_old, v_old = kk.view(torch.int32).cpu().numpy(), vv.view(torch.int32).cpu().numpy()
        kv2 = kv.clone()
        ctx.cast_compact_kv(kk, vv, 3, 3, kk[0].numel() * 4, 2, 64, page, table, wl.seq_capacity(w) // (page or 1),
                            num_pages, apath, alen, kv2)
        assert ctx.cast_poll_status()[0] == 0
        tab = table.cpu().numpy() if table is not None else None
        nk, nv, nlen = compact_kv(k_old, v_old, page, tab, kv.cpu().numpy(), op, ol)
        assert np.array_equal(kv2.cpu().numpy(), nlen)
        assert np.array_equal(kk.view(torch.int32).cpu().numpy(), nk)
        assert np.array_equal(vv.view(torch.int32).cpu().numpy(), nv)


# ------------------------------------------------------------------ acceptance at T > 0
def _run_stochastic(binding, ctx, w, tokens, parent, n_tree, H, T, noise=1.0, inputs=None):
    """GPU against oracle on the same inputs; the oracle's decision margin tells a rounding coin flip
    (pick another seed) from a wrong result."""
    B, Ncap = tokens.shape
    tl, dl, ua, ub = inputs if inputs is not None else wl.stochastic_accept_inputs(w, tokens, parent, n_tree, "cuda", noise, Ncap)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    alen = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    apath = torch.full((B, H + 1), -7, dtype=torch.int32, device="cuda")
    bonus = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ctx.cast_accept_stochastic(tl, dl, B, T, dev(tokens.astype(np.int32)), dev(parent.astype(np.int32)),
                               dev(n_tree.astype(np.int32)), ua, ub, alen, apath, bonus)
    assert ctx.cast_poll_status()[0] == 0
    nmax = int(n_tree.max())
    ol, op, ob, margin = stochastic_accept(to_f64(tl[:, :nmax]), to_f64(dl[:, :nmax]), tokens, parent, n_tree, H, T,
                                           ua.cpu().numpy(), ub.cpu().numpy())
    assert margin.min() >= 1e-9, f"a decision sits within rounding of its threshold ({margin.min():.1e}): pick another seed"
    assert np.array_equal(alen.cpu().numpy(), ol), (alen.cpu().numpy(), ol)
    assert np.array_equal(apath.cpu().numpy(), op), (apath.cpu().numpy(), op)
    assert np.array_equal(bonus.cpu().numpy(), ob), (bonus.cpu().numpy(), ob)
    return ol


def _random_token_tree(rng, B, Ncap, n_tree, V, H, kinds):
    tokens = np.zeros((B, Ncap), dtype=np.int32)
    parent = np.full((B, Ncap), -1, dtype=np.int32)
    for b in range(B):
        N = int(n_tree[b])
        par = _random_tree(rng, N, kinds[b % len(kinds)])
        depth = np.zeros(N, dtype=int)
        for t in range(1, N):
            if depth[par[t]] + 1 > H:  # keep the tree within the depth the output has room for
                par[t] = 0
            depth[t] = depth[par[t]] + 1
        parent[b, :N] = par
        tokens[b, 0] = rng.integers(0, V)
        for t in range(1, N):
            used = {int(tokens[b, c]) for c in range(1, t) if par[c] == par[t]}
            x = int(rng.integers(0, V))
            while x in used:
                x = int(rng.integers(0, V))
            tokens[b, t] = x
    return tokens, parent


@pytest.mark.parametrize("dtype,V,T,B,Ncap,noise", [
    ("f32", 4096, 1.0, 4, 32, 1.0),        # small vocabulary: slices of 256
    ("f32", 1000, 0.7, 3, 32, 0.5),        # slices of 64: the last CTA's slice is short
    ("f32", 37, 1.3, 3, 16, 1.0),          # most CTAs of the cluster hold nothing
    ("bf16", 128256, 1.0, 3, 64, 1.0),     # Llama-3 vocabulary, bf16 logits
    ("f32", 152064, 0.8, 2, 64, 0.3),      # Qwen vocabulary: the largest cached slice
    ("f32", 262144, 1.0, 2, 16, 1.0),      # slices too large to cache: every sweep recomputes them
])
def test_accept_stochastic_random_trees(binding, dtype, V, T, B, Ncap, noise):
    rng = np.random.default_rng(1234 + V)
    H = 6
    w = wl.Workload("sto", 93, B, "f32", dtype, 8, 8, 64, 1, 2, 0, V, 3.0, H, 4, Ncap, False, 1, max_tree=Ncap)
    ctx = binding.CastContext(max_batch=B, vocab=V, top_k=4, max_depth=H, total_token=Ncap, max_tree=Ncap)
    cs, cached = ctx.cast_accept_stochastic_plan(torch.float32 if dtype == "f32" else torch.bfloat16)
    assert cs in (8, 16) and cached == (V <= cs * 12288)
    n_tree = np.array([Ncap, 1, max(2, Ncap // 3), Ncap - 5][:B], dtype=np.int32)
    tokens, parent = _random_token_tree(rng, B, Ncap, n_tree, V, H, ["random", "chain", "star", "random"])
    total = 0
    for rep in range(3):  # three sets of inputs per case: different paths and rejection counts
        w2 = wl.shrink(w, seed_salt=rep)
        total += int(_run_stochastic(binding, ctx, w2, tokens, parent, n_tree, H, T, noise).sum())
    assert total > 0  # the recipe accepts something


def test_accept_stochastic_special_cases(binding):
    rng = np.random.default_rng(77)
    B, Ncap, V, H = 3, 32, 5000, 6
    w = wl.Workload("sto", 94, B, "f32", "f32", 8, 8, 64, 1, 2, 0, V, 3.0, H, 4, Ncap, False, 1, max_tree=Ncap)
    ctx = binding.CastContext(max_batch=B, vocab=V, top_k=4, max_depth=H, total_token=Ncap, max_tree=Ncap)
    n_tree = np.array([Ncap, 20, 9], dtype=np.int32)
    tokens, parent = _random_token_tree(rng, B, Ncap, n_tree, V, H, ["random"])
    tl, dl, ua, ub = wl.stochastic_accept_inputs(w, tokens, parent, n_tree, "cuda", 1.0, Ncap)
    # equal models: the first child is accepted at every node, down to a leaf
    ol = _run_stochastic(binding, ctx, w, tokens, parent, n_tree, H, 1.0, inputs=(dl.clone(), dl, ua, ub))
    for b in range(B):
        cur, steps = 0, 0
        while True:
            kids = [c for c in range(int(n_tree[b])) if parent[b, c] == cur]
            if not kids:
                break
            cur, steps = kids[0], steps + 1
        assert ol[b] == steps
    # a one-hot target: the greedy rule, whatever the uniform numbers are
    hot = tl.clone()
    for b in range(B):
        for t in range(int(n_tree[b])):
            kids = [c for c in range(int(n_tree[b])) if parent[b, c] == t]
            x = int(tokens[b, kids[-1]]) if kids and (t % 3) else int(rng.integers(0, V))
            hot[b, t, x] = 4000.0
    ol = _run_stochastic(binding, ctx, w, tokens, parent, n_tree, H, 1.0, inputs=(hot, dl, ua, ub))
    gl, gp, gb = greedy_accept(to_f64(hot), tokens, parent, n_tree, H)
    assert np.array_equal(ol, gl)
    # what only the device can see goes to the status word: a token outside the vocabulary, a NaN logit
    alen, apath, bonus = (torch.zeros(B, dtype=torch.int32, device="cuda"), torch.zeros((B, H + 1), dtype=torch.int32, device="cuda"),
                          torch.zeros(B, dtype=torch.int32, device="cuda"))
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    bad_tok = tokens.copy()
    bad_tok[1, 1] = V + 5
    ctx.cast_accept_stochastic(tl, dl, B, 1.0, dev(bad_tok), dev(parent), dev(n_tree), ua, ub, alen, apath, bonus)
    assert ctx.cast_poll_status()[0] == 6  # BAD_TREE
    nan_tl = tl.clone()
    nan_tl[2, 0, 17] = float("nan")
    ctx.cast_accept_stochastic(nan_tl, dl, B, 1.0, dev(tokens), dev(parent), dev(n_tree), ua, ub, alen, apath, bonus)
    assert ctx.cast_poll_status()[0] == 8  # NONFINITE
    assert ctx.cast_poll_status()[0] == 0  # the poll cleared it
    # host-side checks
    i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device="cuda")
    for bad_T in (0.0, -1.0, float("nan")):
        with pytest.raises(binding.CastError):
            ctx.cast_accept_stochastic(tl, dl, B, bad_T, i32(B, Ncap), i32(B, Ncap), i32(B), ua, ub, i32(B), i32(B, H + 1), i32(B))
    with pytest.raises(binding.CastError):
        ctx.cast_accept_stochastic(tl, dl, B + 1, 1.0, i32(B, Ncap), i32(B, Ncap), i32(B), ua, ub, i32(B), i32(B, H + 1), i32(B))


# ------------------------------------------------ cost tables measured on the device (Sec. "Method")
def test_measured_cost_tables_size_the_same_tree_on_both_sides(binding):
    """The paper fills S_T(B), S_D(B) by timing the models on the device in use. The profiler here times this
    library's attention over a small (context, tree size) grid on distinct cache buffers, adds the linear
    stand-in for the layer's GEMMs and hands the tables to the library and to the oracle: both must size the
    same tree from them, over two steps, with every sizing switch on."""
    from oracle import CostTable
    from paper_2510_26577_b200 import cost_profile

    B, L, M, Ntab = 2, 256, 3, 24
    w = wl.Workload("prof", 84, B, "bf16", "f32", 8, 2, 128, 40, 600, 16, 3000, 2.0, 5, 4, 20, False, 2, max_tree=32,
                    seed_salt=1)
    t, pts = cost_profile.measure_attention_us(w, B, L, M, n_points=(1, 4, 16, 32), reps=4)
    assert t.shape == (M, 4) and np.isfinite(t).all() and (t > 0).all()
    # a target of 4 layers, a draft head of 1; a GEMM term that makes every further token cost a visible share
    fT, fD = cost_profile.tables_from_measurement(t, pts, B, Ntab, n_layers=4, gemm_us=(5.0, 2.0))
    assert (np.diff(fT, axis=1) > 0).all() and (np.diff(fD, axis=1) > 0).all()
    over = dict(enable_bp=1, enable_dp=1, enable_dr=1, C1=2.0, C2=0.5, C3=0.25)
    kw = cfg_kwargs(w, **over)
    tables = {B: CostTable(B, L, M, Ntab, fT, fD)}
    ctx = binding.CastContext(max_batch=B, **kw)
    ctx.cast_set_cost_tables(B, L, M, Ntab, fT, fD)
    root = wl.root_tokens(w, "cpu").cuda()
    kv = wl.kv_lengths(w, "cpu").cuda()
    oracle = None
    narrowed = False
    for step in range(2):
        logits = [wl.draft_logits(w, 10 * step + l, "cpu", peaked=True).cuda() for l in range(1, w.depth + 1)]
        o = oracle_tree(kw, tables, root, kv, logits, oracle)
        oracle = o["oracle"]
        g = gpu_tree(ctx, root, kv, logits)
        if not (o["min_score_gap"] >= 1e-5 and o["stable"]):
            pytest.skip("a measured table put a decision within rounding of its threshold")
        assert_tree_equal(g, o)
        narrowed |= min(o["n_hist"]) < w.top_k or len(o["n_hist"]) < w.depth or int(o["n_tree"].min()) < w.total_token
    assert narrowed, "the measured tables never narrowed, stopped or trimmed the tree: thresholds out of range"


def test_measured_gemm_terms_give_tables_both_sides_size_alike(binding):
    """The profiler's second measurement: the dense projections of a decoder layer and the vocabulary projection
    at the workload's dimensions (library bf16 GEMMs on random weights). With them the draft's table is no
    longer a multiple of the target's; the library and the oracle, given the same measured tables, must still
    build the same tree with every sizing switch on."""
    from oracle import CostTable
    from paper_2510_26577_b200 import cost_profile

    B, L, M, Ntab = 2, 256, 2, 24
    w = wl.Workload("prof2", 85, B, "bf16", "f32", 8, 2, 128, 40, 400, 16, 3000, 2.0, 4, 4, 16, False, 2, max_tree=32,
                    seed_salt=1)
    pts = (1, 4, 16, 32)
    t, pts = cost_profile.measure_attention_us(w, B, L, M, n_points=pts, reps=4)
    layer_us, head_us = cost_profile.measure_layer_gemms_us(w, B, pts, reps=3)
    assert layer_us.shape == head_us.shape == (len(pts),)
    assert np.isfinite(layer_us).all() and (layer_us > 0).all() and np.isfinite(head_us).all() and (head_us > 0).all()
    fT, fD = cost_profile.tables_from_measurement(t, pts, B, Ntab, n_layers=4, layer_us=layer_us, head_us=head_us)
    assert (np.diff(fT, axis=1) > 0).all() and (np.diff(fD, axis=1) > 0).all()
    over = dict(enable_bp=1, enable_dp=1, enable_dr=1, C1=0.05, C2=0.05, C3=0.02)
    kw = cfg_kwargs(w, **over)
    tables = {B: CostTable(B, L, M, Ntab, fT, fD)}
    ctx = binding.CastContext(max_batch=B, **kw)
    ctx.cast_set_cost_tables(B, L, M, Ntab, fT, fD)
    root = wl.root_tokens(w, "cpu").cuda()
    kv = wl.kv_lengths(w, "cpu").cuda()
    logits = [wl.draft_logits(w, l, "cpu", peaked=True).cuda() for l in range(1, w.depth + 1)]
    o = oracle_tree(kw, tables, root, kv, logits, None)
    g = gpu_tree(ctx, root, kv, logits)
    if not (o["min_score_gap"] >= 1e-5 and o["stable"]):
        pytest.skip("a measured table put a decision within rounding of its threshold")
    assert_tree_equal(g, o)


# ------------------------------------------------ a decoding loop: every step starts from what the last one left
@pytest.mark.parametrize("page", [0, 16])
def test_decoding_loop_of_several_steps(binding, page):
    """Five consecutive steps on one context and one cache, the library and the oracle side by side: tree build
    (all sizing switches on, the FIFO carried along), fresh K/V rows written for the tree tokens right before the
    attention (early reads promised, as in a decoding loop), attention over two layers, greedy acceptance,
    compaction; the next step's root is the bonus token and its prefix the compacted cache. Every output of every
    step is compared, so an error of a step - a row moved to the wrong place, a stale length or work list - shows
    in the same or in a later one."""
    from oracle import CostTable
    B, H, NL = 3, 4, 2
    w = wl.Workload("loop", 90 + (1 if page else 0), B, "bf16", "f32", 8, 2, 128, 60, 500, page, 3000, 2.0, H, 4, 20, True, NL,
                    max_tree=64, seed_salt=2)
    over = dict(enable_dp=1)
    kw = cfg_kwargs(w, **over)
    L, M, Ntab, fT, fD = make_tables(w, B, skewed=True)
    tables = {B: CostTable(B, L, M, Ntab, fT, fD)}
    ctx = binding.CastContext(max_batch=B, **kw)
    ctx.cast_set_cost_tables(B, L, M, Ntab, fT, fD)
    ctx.cast_set_attention_early_reads(True)
    cap = wl.seq_capacity(w)
    table, num_pages = wl.page_table(w, "cuda")
    tab = table.cpu().numpy() if table is not None else None
    layers = [wl.kv_cache(w, l, "cpu") for l in range(NL)]
    kk = torch.stack([k for k, _ in layers]).contiguous().cuda()
    vv = torch.stack([v for _, v in layers]).contiguous().cuda()
    k_ref, v_ref = kk.view(torch.int16).cpu().numpy().copy(), vv.view(torch.int16).cpu().numpy().copy()
    root = wl.root_tokens(w, "cpu").cuda()
    kv = wl.kv_lengths(w, "cpu").cuda()
    kv_ref = kv.cpu().numpy().copy()
    oracle = None
    gen = torch.Generator().manual_seed(w.seed)
    f32 = lambda t: t.float().cpu().numpy()
    bits_to_f32 = lambda a: torch.from_numpy(a).view(torch.bfloat16).float().numpy()
    grew = 0
    for step in range(5):
        logits = [wl.draft_logits(w, 10 * step + l, "cpu", peaked=True).cuda() for l in range(1, H + 1)]
        o = oracle_tree(kw, tables, root, torch.from_numpy(kv_ref), logits, oracle)
        oracle = o["oracle"]
        g = gpu_tree(ctx, root, kv, logits)
        if not (o["min_score_gap"] >= 1e-5 and o["stable"]):
            pytest.skip("a draw put a decision within rounding of its threshold")
        assert_tree_equal(g, o)
        n_tree = o["n_tree"]
        assert (kv_ref + n_tree <= cap).all()
        # the model's K/V rows of the tree tokens, written on both sides at positions L_b .. L_b + N_b - 1
        rows = []
        for b in range(B):
            for t in range(int(n_tree[b])):
                pos = int(kv_ref[b]) + t
                rows.append(int(tab[b, pos // page]) * page + pos % page if page else b * cap + pos)
        idx = torch.tensor(rows, dtype=torch.int64)
        for l in range(NL):
            for cache, ref in ((kk, k_ref), (vv, v_ref)):
                fresh = torch.randn((len(rows), w.kv_heads, w.head_dim), generator=gen).to(torch.bfloat16)
                cache[l].view(-1, w.kv_heads, w.head_dim).index_copy_(0, idx.cuda(), fresh.cuda())
                ref[l].reshape(-1, w.kv_heads, w.head_dim)[rows] = fresh.view(torch.int16).numpy()
        d = g["dev"]
        for l in range(NL):
            q = torch.randn((B, w.max_tree, w.q_heads, w.head_dim), generator=gen).to(torch.bfloat16).cuda()
            out = gpu_attention(ctx, w, q, kk[l], vv[l], table, num_pages, kv, d["anc"], d["n_tree"])
            ref = tree_attention(f32(q), bits_to_f32(k_ref[l]), bits_to_f32(v_ref[l]), page, tab, kv_ref, o["anc"], n_tree)
            got = to_f64(out)
            for b in range(B):
                nb = int(n_tree[b])
                assert np.isnan(got[b, nb:]).all() and np.isfinite(got[b, :nb]).all()
                assert np.max(np.abs(got[b, :nb] - ref[b, :nb])) <= attention_tolerance("bf16"), (step, l, b)
        tl = torch.randn((B, w.max_tree, w.vocab), generator=gen).mul_(2.0).cuda()
        wl.plant_acceptance(w, tl, o["tokens"], o["parent"], n_tree)
        alen = torch.empty((B,), dtype=torch.int32, device="cuda")
        apath = torch.empty((B, H + 1), dtype=torch.int32, device="cuda")
        bonus = torch.empty((B,), dtype=torch.int32, device="cuda")
        ctx.cast_accept(tl, B, d["tokens"], d["parent"], d["depth"], d["anc"], d["n_tree"], alen, apath, bonus)
        nmax = int(n_tree.max())
        ol, op, ob = greedy_accept(to_f64(tl[:, :nmax]), o["tokens"], o["parent"], n_tree, H)
        assert np.array_equal(alen.cpu().numpy(), ol) and np.array_equal(apath.cpu().numpy(), op)
        assert np.array_equal(bonus.cpu().numpy(), ob)
        ctx.cast_compact_kv(kk, vv, B, NL, kk[0].numel() * kk.element_size(), w.kv_heads, w.head_dim, page, table,
                            cap // (page or 1), num_pages, apath, alen, kv)
        assert ctx.cast_poll_status()[0] == 0
        k_ref, v_ref, kv_ref = compact_kv(k_ref, v_ref, page, tab, kv_ref, op, ol)
        assert np.array_equal(kv.cpu().numpy(), kv_ref)
        assert np.array_equal(kk.view(torch.int16).cpu().numpy(), k_ref)
        assert np.array_equal(vv.view(torch.int16).cpu().numpy(), v_ref)
        grew += int(ol.sum())
        root = bonus.clone()
    assert grew >= 5, "the loop accepted almost nothing: the planted acceptances did not take"
    ctx.close()


def test_attention_without_a_reserved_workspace_is_refused(binding):
    """Compute calls never allocate: a shape that needs a split workspace larger than what was reserved
    returns CAST_ERR_CAPACITY and launches nothing; after cast_reserve_attention the same call runs."""
    w = wl.shrink(wl.CONFIGS["c1_tiny"])
    ctx = binding.CastContext(max_batch=1, **cfg_kwargs(w))
    q = wl.query(w, 0, "cuda")
    k, v = wl.kv_cache(w, 0, "cuda")
    kv = wl.kv_lengths(w, "cuda")
    anc = torch.zeros((1, w.max_tree, ctx.words), dtype=torch.int32, device="cuda")
    anc[0, 0, 0] = 1
    nt = torch.ones(1, dtype=torch.int32, device="cuda")
    out = torch.full_like(q, float("nan"))
    args = (q, k, v, 1, w.q_heads, w.kv_heads, w.head_dim, 0, None, wl.seq_capacity(w), 0, kv, anc, nt, 0.0, out)
    with pytest.raises(binding.CastError) as e:
        ctx.cast_tree_attention(*args)
    assert e.value.code == 3
    torch.cuda.synchronize()
    assert torch.isnan(out).all()
    free0 = torch.cuda.mem_get_info()[0]
    ctx.cast_reserve_attention(q.dtype, 1, w.q_heads, w.kv_heads, w.head_dim, 0, wl.seq_capacity(w))
    free1 = torch.cuda.mem_get_info()[0]
    ctx.cast_tree_attention(*args)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free1 <= free0  # the compute call moved no device memory
    assert torch.isfinite(out[0, 0]).all() and ctx.cast_poll_status()[0] == 0


# ------------------------------------------------ the seeds the benchmark configurations pass over
@pytest.mark.parametrize("name,salt", [("c3_llama8b_b1", 0), ("c3_llama8b_b1", 1), ("c5_qwen_long", 0), ("c3_llama8b_b64", 0)])
def test_seeds_passed_over_for_their_margin_still_match(binding, name, salt):
    """A configuration's seed_salt skips seeds on which the ORACLE has a decision within rounding of its
    threshold (a gap below 1e-5 between neighbouring values, or a test that flips under a relative 2e-6):
    there a bit-exact comparison with fp32 device arithmetic is not well posed. They were not skipped because
    the device disagreed: on these seeds it builds the oracle's tree as well (tests/seed_margin_audit.py lists
    the margins; the smallest gap here is 5e-6)."""
    w = wl.shrink(wl.CONFIGS[name], seed_salt=salt)
    kw = cfg_kwargs(w)
    B = w.batch
    tables, raw = _oracle_tables(w, B) if w.cost_model else (None, None)
    ctx = binding.CastContext(max_batch=B, **kw)
    if raw is not None:
        ctx.cast_set_cost_tables(B, *raw)
    root = wl.root_tokens(w, "cpu").cuda()
    kv = wl.kv_lengths(w, "cpu").cuda()
    logits = [wl.draft_logits(w, l, "cpu").cuda() for l in range(1, w.depth + 1)]
    o = oracle_tree(kw, tables, root, kv, logits)
    assert not (o["min_score_gap"] >= 1e-5 and o["stable"]), "this seed is not a marginal one any more"
    g = gpu_tree(ctx, root, kv, logits)
    print(f"{name} salt {salt}: oracle gap {o['min_score_gap']:.2e}, stable {o['stable']}")
    assert_tree_equal(g, o)


# ------------------------------------------------ attention with early reads (the caller's promise)
@pytest.mark.parametrize("name", ["c2_llama8b", "c3_llama8b_b4", "c3_llama8b_b16", "c4_llama70b_n32"])
def test_attention_early_reads_give_the_same_bits(binding, name):
    """With cast_set_attention_early_reads the kernel decodes its work, reads the masks and fetches prefix tiles
    before its predecessor on the stream has finished. Two whole steps (tree build, four attention layers back
    to back on different caches, acceptance, compaction - which moves kv_len and cache rows that the next step's
    attention reads) run without any host synchronisation in between, once per mode: every attention output,
    the accepted paths and the lengths must be bit-identical to the default mode's, which the tests above
    compare with the oracle."""
    w = wl.CONFIGS[name]
    B, H, nl = w.batch, w.depth, 4
    kw = cfg_kwargs(w)
    tabs = wl.cost_table_arrays(w, B) if w.cost_model else None
    root = wl.root_tokens(w, "cpu").cuda()
    kv0 = wl.kv_lengths(w, "cpu").cuda()
    logits = [[wl.draft_logits(w, 10 * s_ + l, "cuda") for l in range(1, H + 1)] for s_ in range(2)]
    q = [wl.query(w, l, "cuda") for l in range(nl)]
    table, num_pages = wl.page_table(w, "cuda")
    seq_cap = wl.seq_capacity(w) // (w.page_size or 1)
    tl = wl.target_logits(w, "cuda")
    results = []
    for promise in (False, True):
        ctx = binding.CastContext(max_batch=B, **kw)
        if tabs is not None:
            ctx.cast_set_cost_tables(B, *tabs)
        ctx.cast_reserve_attention(q[0].dtype, B, w.q_heads, w.kv_heads, w.head_dim, w.page_size, seq_cap)
        ctx.cast_set_attention_early_reads(promise)
        kc = torch.stack([wl.kv_cache(w, l, "cuda")[0] for l in range(nl)]).contiguous()
        vc = torch.stack([wl.kv_cache(w, l, "cuda")[1] for l in range(nl)]).contiguous()
        kv = kv0.clone()
        tr = alloc_tree_outputs(B, w.max_tree, ctx.words)
        nt = torch.empty((B, w.top_k), dtype=torch.int32, device="cuda")
        npr, cnt = torch.empty_like(nt), torch.empty((1,), dtype=torch.int32, device="cuda")
        alen = torch.empty((B,), dtype=torch.int32, device="cuda")
        apath = torch.empty((B, H + 1), dtype=torch.int32, device="cuda")
        bonus = torch.empty((B,), dtype=torch.int32, device="cuda")
        outs = []
        for s_ in range(2):
            ctx.cast_step_begin(B, root, kv)
            for i in range(H):
                ctx.cast_tree_expand(i + 1, logits[s_][i], nt, npr, cnt)
            ctx.cast_select_nodes(tr["tokens"], tr["parent"], tr["depth"], tr["anc"], tr["pool_idx"], tr["scores"], tr["n_tree"])
            for l in range(nl):
                out = torch.full_like(q[l], float("nan"))
                ctx.cast_tree_attention(q[l], kc[l], vc[l], B, w.q_heads, w.kv_heads, w.head_dim, w.page_size, table, seq_cap,
                                        num_pages, kv, tr["anc"], tr["n_tree"], 0.0, out)
                outs.append(out)
            ctx.cast_accept(tl, B, tr["tokens"], tr["parent"], tr["depth"], tr["anc"], tr["n_tree"], alen, apath, bonus)
            ctx.cast_compact_kv(kc, vc, B, nl, kc[0].numel() * kc.element_size(), w.kv_heads, w.head_dim, w.page_size, table,
                                seq_cap, num_pages, apath, alen, kv)
            outs += [alen.clone(), apath.clone(), kv.clone()]
        torch.cuda.synchronize()
        assert ctx.cast_poll_status()[0] == 0
        results.append([o.view(torch.int16) if o.dtype == torch.bfloat16 else o for o in outs] + [kc.view(torch.int16), vc.view(torch.int16)])
    for a, b2 in zip(*results):
        assert torch.equal(a, b2)
    assert int(results[0][-3].min()) > int(kv0.min())  # the compaction did advance the lengths
