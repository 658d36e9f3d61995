"""Benchmark of the CAST draft-and-verify step on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input:
cast_step_begin, H x cast_tree_expand, cast_select_nodes, n_layers x
cast_tree_attention (distinct KV buffers per layer), cast_accept,
cast_compact_kv - captured in one CUDA graph and replayed.  The headline value
is tree tokens verified per second; the per-phase timings, the attention
roofline and the CPU oracle baseline ride along in the same JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
  python bench.py --impl reference ...      (the CPU oracle, bounded sample)
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC, UNIT = "tree_verify_tokens_per_s", "tokens/s"

# DRAM bytes (read + write) of one tree_attn_tc_kernel launch from the ncu captures summarised
# under profiles/ (same launch shape as one layer of the workload).
NCU_ATTENTION_TRAFFIC = {"c2_llama8b": 9.29e6, "c3_llama8b_b16": 144.8e6, "c3_llama8b_b64": 598.4e6,
                         "c4_llama70b_n128": 179.5e6}


NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0  # what the hardware's data sheet says (context only)


def peaks():
    """(HBM GB/s, sustained dense bf16 TFLOP/s, source): the measured figures of this machine, else the
    stated fallback. The attention launches are timed inside a long graph, hence the sustained GEMM figure."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", d.get("bf16_tflops", 1400.0))), "measured"
    return 6650.0, 1400.0, "fallback"


def static_config(w, tokens_per_step, world):
    """The workload description both arms print (same keys, same values)."""
    return {"workload": w.name, "batch": w.batch, "tree_tokens_per_step": tokens_per_step, "depth": w.depth,
            "top_k": w.top_k, "vocab": w.vocab, "q_heads": w.q_heads, "kv_heads": w.kv_heads, "head_dim": w.head_dim,
            "kv_prefix": [w.kv_len_lo, w.kv_len_hi], "page_size": w.page_size, "n_layers": w.n_layers,
            "kv_dtype": w.kv_dtype, "logit_dtype": w.logit_dtype,
            "parallelism": "replicas" if world > 1 else "single"}


class ClockSampler:
    """SM clock and throttle reasons read through NVML every few milliseconds by a thread,
    from just before the timed region to just after it (reading only: nothing is set)."""
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.002):
        import threading
        self.samples, self.mask, self.max_mhz, self.power = [], 0, None, []
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            ids = [x.strip() for x in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if x.strip()]
            if ids and index < len(ids):  # NVML numbers all GPUs of the host; CUDA only the visible ones
                tok = ids[index]
                self.h = (pynvml.nvmlDeviceGetHandleByIndex(int(tok)) if tok.isdigit()
                          else pynvml.nvmlDeviceGetHandleByUUID(tok))
            else:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.nv = pynvml
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None
            return

        def loop():
            nv = self.nv
            while not self._stop.is_set():
                try:
                    self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                    self.mask |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                except Exception:
                    pass
                self._stop.wait(period_s)

        self._thread = threading.Thread(target=loop, daemon=True)
        self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join(timeout=2)
        sm = self.samples
        reasons = sorted(n for n, bit in self.REASONS.items() if self.mask & bit)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(sm), "power_w_max": max(self.power) if self.power else None}


# ------------------------------------------------------------------ CPU oracle arm
def oracle_step_seconds(w, attn_pairs=256):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload and
    extrapolates to one full step.  Returns (seconds_per_step, description, threads)."""
    import numpy as np
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import cfg_kwargs, make_tables, oracle_tree, to_f64
    from oracle import CostTable, compact_kv, greedy_accept, tree_attention
    from paper_2510_26577_b200 import workloads as wl

    kw = cfg_kwargs(w)
    B = w.batch
    tables = None
    if w.cost_model:
        L, M, Ntab, fT, fD = make_tables(w, B)
        tables = {B: CostTable(B, L, M, Ntab, fT, fD)}
    root, kv = wl.root_tokens(w), wl.kv_lengths(w)
    logits = [wl.draft_logits(w, l) for l in range(1, w.depth + 1)]
    t0 = time.perf_counter()
    o = oracle_tree(kw, tables, root, kv, logits)
    t_tree = time.perf_counter() - t0
    n_tree = o["n_tree"]
    q = wl.query(w, 0).float().numpy()
    k, v = (t.float().numpy() for t in wl.kv_cache(w, 0))
    table, _ = wl.page_table(w)
    tab = table.numpy() if table is not None else None
    rng = np.random.default_rng(0)
    total_pairs = int(sum(int(n) for n in n_tree)) * w.q_heads
    only = set()
    while len(only) < min(attn_pairs, total_pairs):
        b = int(rng.integers(0, B))
        only.add((b, int(rng.integers(0, n_tree[b])), int(rng.integers(0, w.q_heads))))
    t0 = time.perf_counter()
    tree_attention(q, k, v, w.page_size, tab, kv.numpy(), o["anc"], n_tree, None, only)
    t_attn_layer = (time.perf_counter() - t0) * total_pairs / len(only)
    nmax = int(n_tree.max())
    tl = to_f64(wl.target_logits(w)[:, :nmax])
    t0 = time.perf_counter()
    ol, op, _ = greedy_accept(tl, o["tokens"], o["parent"], n_tree, w.depth)
    t_accept = time.perf_counter() - t0
    kk, vv = k[None], v[None]
    t0 = time.perf_counter()
    compact_kv(kk, vv, w.page_size, tab, kv.numpy(), op, ol)
    t_compact = (time.perf_counter() - t0) * w.n_layers
    total = t_tree + w.n_layers * t_attn_layer + t_accept + t_compact
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = 1
    desc = (f"tree build + accept in full; attention: {len(only)} of {total_pairs} (token, head) outputs of one layer, "
            f"scaled to {w.n_layers} layers; compaction of one layer scaled to {w.n_layers}")
    return total, desc, threads, int(sum(int(n) for n in n_tree)), float(ol.mean())


def run_reference(args, w):
    """The oracle on the host cores. A step here is a bounded sample of the workload's step (tree build and
    accept in full, a sample of one layer's attention outputs, one layer's compaction); `ms_per_step` is what
    that sample took, `value` the whole-step throughput it extrapolates to."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times, walls = [], []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        sec, desc, threads, ntok, acc_mean = oracle_step_seconds(w, attn_pairs=64)
        if i >= args.warmup:
            times.append(sec)
            walls.append(time.perf_counter() - t0)
    sec = sum(times) / len(times)
    val = ntok / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sum(walls) / len(walls) * 1e3, "ms_per_full_step_extrapolated": sec * 1e3,
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": static_config(w, ntok, args.gpus),
        "timing": {"accept_len_mean": acc_mean},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------ CUDA arm
def measure(args, w, rep, full):
    """Builds the workload's inputs on the device, times the step and its phases. `full`: the headline
    workload (all phases, end-to-end leg, CPU baseline); otherwise a short pass for the workloads table."""
    import numpy as np
    import torch
    from paper_2510_26577_b200 import binding, replicas, workloads as wl

    rank, world = rep.rank, rep.world
    local = rep.local_rank
    dev = torch.device("cuda", local)
    quick = args.quick or not full

    B, H, K, Ncap, m = w.batch, w.depth, w.top_k, w.max_tree, w.total_token
    Hq, Hkv, D, nl = w.q_heads, w.kv_heads, w.head_dim, w.n_layers
    kw = dict(vocab=w.vocab, top_k=K, max_depth=H, total_token=m, max_tree=Ncap)
    if w.cost_model:
        kw.update(enable_bp=1, enable_dr=1)
    ctx = binding.CastContext(max_batch=B, **kw)
    if w.cost_model:
        ctx.cast_set_cost_tables(B, *wl.cost_table_arrays(w, B))
    seq_cap = wl.seq_capacity(w) // (w.page_size or 1)
    ctx.cast_reserve_attention(torch.bfloat16 if w.kv_dtype == "bf16" else torch.float32, B, Hq, Hkv, D, w.page_size,
                               seq_cap)
    # a decoding loop: between two attention layers nothing writes the tree, the lengths or the prefix rows
    ctx.cast_set_attention_early_reads(True)
    l2_bytes = int(torch.cuda.get_device_properties(dev).L2_cache_size)

    # ---- synthetic inputs, resident in HBM
    root, kv0 = wl.root_tokens(w, dev), wl.kv_lengths(w, dev)
    kv_len = kv0.clone()
    logits = [wl.draft_logits(w, l, dev) for l in range(1, H + 1)]
    q = torch.stack([wl.query(w, l, dev) for l in range(nl)])
    kc = torch.empty((nl,) + tuple(wl.kv_cache(w, 0, dev)[0].shape), dtype=q.dtype, device=dev)
    vc = torch.empty_like(kc)
    for l in range(nl):
        kc[l], vc[l] = wl.kv_cache(w, l, dev)
    table, num_pages = wl.page_table(w, dev)
    tl = wl.target_logits(w, dev)
    out = torch.zeros_like(q)
    nt = [torch.empty((B, K), dtype=torch.int32, device=dev) for _ in range(H)]
    npr = [torch.empty((B, K), dtype=torch.int32, device=dev) for _ in range(H)]
    cnt = [torch.empty((1,), dtype=torch.int32, device=dev) for _ in range(H)]
    tr = dict(tokens=torch.empty((B, Ncap), dtype=torch.int32, device=dev),
              parent=torch.empty((B, Ncap), dtype=torch.int32, device=dev),
              depth=torch.empty((B, Ncap), dtype=torch.int32, device=dev),
              anc=torch.empty((B, Ncap, ctx.words), dtype=torch.int32, device=dev),
              pool_idx=torch.empty((B, Ncap), dtype=torch.int32, device=dev),
              scores=torch.empty((B, Ncap), dtype=torch.float64, device=dev),
              n_tree=torch.empty((B,), dtype=torch.int32, device=dev))
    alen = torch.empty((B,), dtype=torch.int32, device=dev)
    apath = torch.empty((B, H + 1), dtype=torch.int32, device=dev)
    bonus = torch.empty((B,), dtype=torch.int32, device=dev)
    layer_stride = kc[0].numel() * kc.element_size()

    def tree_build(lg=None):
        lg = lg or logits
        ctx.cast_step_begin(B, root, kv_len)
        for i in range(H):
            ctx.cast_tree_expand(i + 1, lg[i], nt[i], npr[i], cnt[i])
        ctx.cast_select_nodes(tr["tokens"], tr["parent"], tr["depth"], tr["anc"], tr["pool_idx"], tr["scores"],
                              tr["n_tree"])

    def attention():
        for l in range(nl):
            ctx.cast_tree_attention(q[l], kc[l], vc[l], B, Hq, Hkv, D, w.page_size, table, seq_cap, num_pages, kv_len,
                                    tr["anc"], tr["n_tree"], 0.0, out[l])

    def accept(t=None):
        ctx.cast_accept(tl if t is None else t, B, tr["tokens"], tr["parent"], tr["depth"], tr["anc"], tr["n_tree"],
                        alen, apath, bonus)

    def compact():
        ctx.cast_compact_kv(kc, vc, B, nl, layer_stride, Hkv, D, w.page_size, table, seq_cap, num_pages, apath, alen,
                            kv_len)

    def step():
        kv_len.copy_(kv0)  # compaction advanced the lengths; every step starts from the same prefix
        tree_build(); attention(); accept(); compact()

    # first pass: gives the tree for planting acceptance
    tree_build()
    torch.cuda.synchronize()
    st, detail = ctx.cast_poll_status()
    assert st == 0, f"device status {st} ({detail})"
    n_tree = tr["n_tree"].cpu().numpy()
    n_hist = ctx.cast_step_info()["n_hist"]
    wl.plant_acceptance(w, tl, tr["tokens"].cpu().numpy(), tr["parent"].cpu().numpy(), n_tree)
    step()
    torch.cuda.synchronize()
    assert ctx.cast_poll_status()[0] == 0
    tokens_per_step = int(n_tree.sum())
    accept_mean = float(alen.float().mean().item())

    stream = torch.cuda.Stream(device=dev)

    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            kv_len.copy_(kv0)  # an earlier pass may have run the compaction
            fn()  # warm the stream
            kv_len.copy_(kv0)
            stream.synchronize()
            with torch.cuda.graph(g, stream=stream):
                fn()
        return g

    def time_graph(g, reps, warm):
        with torch.cuda.stream(stream):
            for _ in range(warm):
                g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            stream.synchronize()
            e0.record(stream)
            for _ in range(reps):
                g.replay()
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) / reps  # ms per replay

    def make_accept_stochastic():
        """Acceptance at temperature 1 on the step's tree: inputs (two more [B, Ncap, V] logit tensors) and call."""
        s_tl, s_dl, s_ua, s_ub = wl.stochastic_accept_inputs(w, tr["tokens"].cpu().numpy(), tr["parent"].cpu().numpy(),
                                                             n_tree, dev, 0.7, Ncap)
        s_len = torch.empty_like(alen)
        s_path, s_bonus = torch.empty_like(apath), torch.empty_like(bonus)

        def call():
            ctx.cast_accept_stochastic(s_tl, s_dl, B, 1.0, tr["tokens"], tr["parent"], tr["n_tree"], s_ua, s_ub, s_len,
                                       s_path, s_bonus)
        return call, s_len, s_tl.dtype

    if args.only:  # profiling aid: replay one phase only (no graph), print its time, stop
        if args.only == "accept_stochastic":
            fn = make_accept_stochastic()[0]
        else:
            fn = {"tree": tree_build, "attention": attention, "accept": accept, "compact": compact}[args.only]
        with torch.cuda.stream(stream):
            kv_len.copy_(kv0)  # the first pass ran the compaction
            for _ in range(args.warmup):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                if args.only == "compact":
                    kv_len.copy_(kv0)
                fn()
            e1.record(stream)
            stream.synchronize()
        st = ctx.cast_poll_status()
        print(json.dumps({"only": args.only, "workload": w.name, "us_per_call": e0.elapsed_time(e1) * 1e3 / args.steps,
                          "device_status": st[0]}))
        return None

    g_step = capture(step)

    def compact_phase():
        kv_len.copy_(kv0)  # each replay compacts from the same prefix lengths
        compact()

    # Phases timed alone read their inputs cold, like the step does (there the KV traffic of the attention
    # layers evicts the logits between two steps): the phase graph walks through copies of its logits at
    # different addresses, more than twice the L2 in total, before it comes back to the first.
    esz = logits[0].element_size()
    draft_bytes = sum(B * (n_hist[i - 1] if i > 0 else 1) * w.vocab * esz for i in range(H) if i == 0 or n_hist[i - 1] > 0)
    target_bytes = int(n_tree.sum()) * w.vocab * tl.element_size()

    def copies_for(nbytes):
        return 1 if nbytes >= 2 * l2_bytes else min(-(-2 * l2_bytes // max(nbytes, 1)) + 1, 24)

    n_dsets, n_tsets = copies_for(draft_bytes), copies_for(target_bytes)
    dsets = [logits] + [[x.clone() for x in logits] for _ in range(n_dsets - 1)]
    tsets = [tl] + [tl.clone() for _ in range(n_tsets - 1)]

    def tree_build_phase():
        for lg in dsets:
            tree_build(lg)

    def accept_phase():
        for t in tsets:
            accept(t)

    g_tree, g_attn, g_acc, g_cmp = capture(tree_build_phase), capture(attention), capture(accept_phase), capture(compact_phase)

    # acceptance at temperature 1 on the same tree (not part of the step: it replaces cast_accept when the
    # serving loop samples). Its inputs hold two more [B, Ncap, V] logit tensors: skipped above 2^28 entries.
    sto = None
    if B * Ncap * w.vocab <= (1 << 28) and not quick:
        accept_stochastic, s_len, s_dtype = make_accept_stochastic()
        ms_sto = time_graph(capture(accept_stochastic), max(args.steps, 20), args.warmup)
        plan = ctx.cast_accept_stochastic_plan(s_dtype)
        sto = {"us": ms_sto * 1e3, "temperature": 1.0, "target_minus_draft_logit_std": 0.7,
               "mean_accept_len": float(s_len.float().mean().item()), "cluster_size": plan[0], "slices_cached": plan[1]}
        del accept_stochastic

    # the draft-side use of the attention kernel: layer by layer, the new layer's tokens against the prefix
    # and the earlier layers (rows of the growing tree); one verification layer's KV buffer per call
    dep = tr["depth"].cpu().numpy()
    windows = []
    for d_ in range(1, H + 1):
        first = np.array([int(np.sum(dep[b_, : n_tree[b_]] < d_)) for b_ in range(B)], dtype=np.int32)
        end = np.array([int(np.sum(dep[b_, : n_tree[b_]] <= d_)) for b_ in range(B)], dtype=np.int32)
        if int((end - first).sum()) > 0:
            windows.append((torch.from_numpy(first).to(dev), torch.from_numpy(end).to(dev)))

    def draft_attention():
        for i_, (first, end) in enumerate(windows):
            l_ = i_ % nl
            ctx.cast_tree_attention_rows(q[l_], kc[l_], vc[l_], B, Hq, Hkv, D, w.page_size, table, seq_cap, num_pages,
                                         kv_len, tr["anc"], end, first, 0.0, out[l_])

    draft_attn_us = None
    if windows and not quick:
        draft_attn_us = time_graph(capture(draft_attention), max(args.steps, 20), args.warmup) * 1e3 / len(windows)

    # ---- phase timings (each phase alone; every phase's working set exceeds 2x L2 between reuses)
    kv_len.copy_(kv0)  # the capture passes ran the compaction
    sub_reps = max(args.steps // 2, 5) if quick else max(args.steps, 20)
    warm = max(args.warmup, 3)
    ms_tree = time_graph(g_tree, sub_reps, warm) / n_dsets
    ms_attn = time_graph(g_attn, sub_reps, warm)
    ms_acc = time_graph(g_acc, sub_reps, warm) / n_tsets
    ms_cmp = time_graph(g_cmp, sub_reps, warm)
    kv_len.copy_(kv0)
    del dsets, tsets, g_tree, g_acc

    # ---- the timed region: K replays of the whole step
    replicas.barrier(rep)
    torch.cuda.synchronize()
    sampler = ClockSampler(local) if rank == 0 else None
    ms_step = time_graph(g_step, args.steps if full else max(args.steps // 2, 5), warm)
    total_tokens, ms_step = replicas.aggregate(rep, tokens_per_step, ms_step)
    replicas.barrier(rep)
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    st = ctx.cast_poll_status()
    assert st[0] == 0, f"device status {st}"

    # ---- roofline of the dominant kernel (tree attention, one layer per launch): which roof applies follows
    # from the launch's arithmetic intensity (4 D rows flop per position and kv-head against 2 D e bytes)
    e = 2 if w.kv_dtype == "bf16" else 4
    kvl = kv0.cpu().numpy().astype(np.int64)
    G = Hq // Hkv
    attn_bytes = int(sum(2 * (int(kvl[b]) + int(n_tree[b])) * Hkv * D * e + 2 * int(n_tree[b]) * Hq * D * e
                         for b in range(B)))
    attn_flops = int(sum(4 * D * int(n_tree[b]) * G * Hkv * (int(kvl[b]) + int(n_tree[b])) for b in range(B)))
    hbm_peak, tensor_peak, which = peaks()
    attn_us = ms_attn * 1e3 / nl
    tensor_path = w.kv_dtype == "bf16" and D == 128
    ridge = tensor_peak * 1e12 / (hbm_peak * 1e9)
    gbs = attn_bytes / (attn_us * 1e-6) / 1e9
    tfs = attn_flops / (attn_us * 1e-6) / 1e12
    if tensor_path and attn_flops / attn_bytes > 1.1 * ridge:  # within 10 % of the ridge the HBM roof is the one reported
        roof = {"kernel": "cast_tree_attention (one layer)", "bound": "tensor", "achieved": tfs, "peak": tensor_peak,
                "unit": "TFLOP/s", "frac": tfs / tensor_peak, "frac_of_nominal": tfs / NOMINAL_BF16_TFLOPS,
                "peak_source": which + " (sustained bf16 GEMM)", "traffic": NCU_ATTENTION_TRAFFIC.get(w.name),
                "algorithmic_flops": attn_flops, "algorithmic_bytes": attn_bytes, "hbm_gbs": gbs}
    else:
        roof = {"kernel": "cast_tree_attention (one layer)", "bound": "hbm", "achieved": gbs, "peak": hbm_peak,
                "unit": "GB/s", "frac": gbs / hbm_peak, "frac_of_nominal": gbs / NOMINAL_HBM_GBS, "peak_source": which,
                "traffic": NCU_ATTENTION_TRAFFIC.get(w.name), "algorithmic_bytes": attn_bytes,
                "algorithmic_flops": attn_flops, "tensor_tflops": tfs if tensor_path else None}
    roof["flop_per_byte"] = attn_flops / attn_bytes
    roof["ridge_flop_per_byte"] = ridge
    # the two vocabulary sweeps against the HBM roof: logits read once per row (cold)
    sweeps = {
        "tree_build": {"kernel": "cast_step_begin + H x cast_tree_expand + cast_select_nodes", "bound": "hbm",
                       "algorithmic_bytes": int(draft_bytes), "us": ms_tree * 1e3,
                       "achieved": draft_bytes / (ms_tree * 1e-3) / 1e9, "peak": hbm_peak, "unit": "GB/s",
                       "frac": draft_bytes / (ms_tree * 1e-3) / 1e9 / hbm_peak, "logit_copies_rotated": n_dsets},
        "accept": {"kernel": "cast_accept (argmax sweep + walk)", "bound": "hbm", "algorithmic_bytes": int(target_bytes),
                   "us": ms_acc * 1e3, "achieved": target_bytes / (ms_acc * 1e-3) / 1e9, "peak": hbm_peak,
                   "unit": "GB/s", "frac": target_bytes / (ms_acc * 1e-3) / 1e9 / hbm_peak,
                   "logit_copies_rotated": n_tsets},
    }
    sel_launches = 1 if B == 1 else 2
    attn_launches = 1 if tensor_path else 2  # CUDA-core path: main + combine
    # H expand + select + attention layers (+ the work-list kernel in front of the first one) + sweep, walk + compaction
    launches_per_step = H + sel_launches + attn_launches * nl + (1 if tensor_path else 0) + 2 + 1
    res = {
        "w": w, "tokens_per_step": tokens_per_step, "total_tokens": total_tokens, "ms_step": ms_step, "clocks": clocks,
        "accept_mean": accept_mean, "launches_per_step": launches_per_step, "roofline": roof, "sweeps": sweeps,
        "phases": {"tree_build_us": ms_tree * 1e3, "attention_us_per_layer": attn_us, "accept_us": ms_acc * 1e3,
                   "compact_us": ms_cmp * 1e3, "accept_stochastic": sto, "draft_attention_us_per_layer": draft_attn_us},
        "n_hist": [int(x) for x in n_hist[:H]], "n_tree": [int(x) for x in n_tree],
    }
    if not full:
        return res

    # ---- end to end: every step's inputs start in pinned host memory and its results are read back to
    # the host, all inside the timed region. Uploads and downloads run on a stream each into / out of a
    # second set of device buffers, so the upload of step s+1 overlaps the compute of step s and the
    # download of step s-1 (PCIe, which carries both directions at once, is the bound).
    # One pinned arena holds a step's inputs and one its results, so that each direction is one copy per step
    # (eight separate copies reached 51 GB/s on this link, one 54).
    srcs = [x for x in logits] + [q[:, :, :m].contiguous(), tl[:, :m].contiguous()]

    def carve(arena, like):  # views of the tensors' shapes and types at 256-byte steps of a byte arena
        views, off = [], 0
        for x in like:
            nbytes = x.numel() * x.element_size()
            views.append(arena[off:off + nbytes].view(x.dtype).view(x.shape))
            off += (nbytes + 255) // 256 * 256
        return views

    in_bytes = sum((x.numel() * x.element_size() + 255) // 256 * 256 for x in srcs)
    h_in = torch.empty(in_bytes, dtype=torch.uint8).pin_memory()
    for v, x in zip(carve(h_in, srcs), srcs):
        v.copy_(x)
    res_like = [srcs[H], torch.empty((B, H + 3), dtype=torch.int32)]
    out_bytes = sum((x.numel() * x.element_size() + 255) // 256 * 256 for x in res_like)
    h_res_arena = torch.empty(out_bytes, dtype=torch.uint8).pin_memory()
    h2d = sum(x.numel() * x.element_size() for x in srcs)
    d2h = sum(x.numel() * x.element_size() for x in res_like)
    copy_stream = torch.cuda.Stream(device=dev)
    down_stream = torch.cuda.Stream(device=dev)
    stage_in_arena = [torch.empty(in_bytes, dtype=torch.uint8, device=dev) for _ in range(2)]
    stage_out_arena = [torch.empty(out_bytes, dtype=torch.uint8, device=dev) for _ in range(2)]
    stage_in, stage_out = [], []
    for k in range(2):
        v = carve(stage_in_arena[k], srcs)
        stage_in.append(dict(logits=v[:H], q=v[H], tl=v[H + 1]))
        v = carve(stage_out_arena[k], res_like)
        stage_out.append(dict(out=v[0], res=v[1]))
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]
    ev_free = [torch.cuda.Event() for _ in range(2)]
    ev_down = [torch.cuda.Event() for _ in range(2)]

    def upload(k):  # copy stream: host -> staging set k
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(ev_free[k])  # the compute stream has taken the previous contents
            stage_in_arena[k].copy_(h_in, non_blocking=True)
            ev_in[k].record(copy_stream)

    def compute(k):  # compute stream: staging set k -> the graph's inputs, one step, results -> staging set k
        with torch.cuda.stream(stream):
            stream.wait_event(ev_in[k])
            for i in range(H):
                logits[i].copy_(stage_in[k]["logits"][i], non_blocking=True)
            q[:, :, :m].copy_(stage_in[k]["q"], non_blocking=True)
            tl[:, :m].copy_(stage_in[k]["tl"], non_blocking=True)
            ev_free[k].record(stream)
            g_step.replay()
            stream.wait_event(ev_down[k])  # the previous results of this set have reached the host
            stage_out[k]["out"].copy_(out[:, :, :m], non_blocking=True)
            r = stage_out[k]["res"]
            r[:, 0] = alen; r[:, 1] = bonus; r[:, 2:] = apath
            ev_out[k].record(stream)

    def download(k):  # download stream: results of staging set k -> host
        with torch.cuda.stream(down_stream):
            down_stream.wait_event(ev_out[k])
            h_res_arena.copy_(stage_out_arena[k], non_blocking=True)
            ev_down[k].record(down_stream)

    def e2e_run(nsteps):
        for k in range(2):
            ev_free[k].record(stream)
            ev_down[k].record(down_stream)
        upload(0)
        for sidx in range(nsteps):
            k = sidx & 1
            if sidx + 1 < nsteps:
                upload(k ^ 1)
            compute(k)
            download(k)
        copy_stream.synchronize()
        down_stream.synchronize()
        stream.synchronize()

    e2e_steps = 2 if args.quick else args.steps
    if not args.quick:
        e2e_run(max(args.warmup, 3))
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    e2e_run(e2e_steps)
    e1.record(stream)
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    ms_e2e = max(e0.elapsed_time(e1) / e2e_steps, wall_ms)  # the copy stream may finish after the compute stream
    _, ms_e2e = replicas.aggregate(rep, tokens_per_step, ms_e2e)
    res["e2e"] = {"value": total_tokens / (ms_e2e * 1e-3), "unit": UNIT, "ms_per_step": ms_e2e,
                  "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)}
    return res


# Workloads of the table that rides along with the headline (every benchmark configuration), each
# measured by a short pass: few replays, no end-to-end leg, no CPU baseline.
TABLE_WORKLOADS = ["c1_tiny", "c3_llama8b_b1", "c3_llama8b_b4", "c3_llama8b_b16", "c3_llama8b_b64", "c4_llama70b_n16",
                   "c4_llama70b_n32", "c4_llama70b_n64", "c4_llama70b_n128", "c5_qwen_long"]


def table_row(r):
    roof, ph, w = r["roofline"], r["phases"], r["w"]
    ck = r["clocks"] or {}
    return {"workload": w.name, "batch": w.batch, "n_layers": w.n_layers, "tree_tokens_per_step": r["tokens_per_step"],
            "n_per_layer": r["n_hist"], "ms_per_step": round(r["ms_step"], 4),
            "tokens_per_s": round(r["tokens_per_step"] / (r["ms_step"] * 1e-3), 1),
            "tree_build_us": round(ph["tree_build_us"], 2), "attention_us_per_layer": round(ph["attention_us_per_layer"], 2),
            "accept_us": round(ph["accept_us"], 2), "compact_us": round(ph["compact_us"], 2),
            "bound": roof["bound"], "achieved": round(roof["achieved"], 1), "unit": roof["unit"],
            "frac": round(roof["frac"], 4), "hbm_gbs": round(roof.get("hbm_gbs", roof["achieved"]), 1),
            "sm_mhz": ck.get("sm_mhz"), "reasons": ck.get("reasons")}


def run_ours(args, w):
    import gc
    import torch
    from paper_2510_26577_b200 import build as _build
    _build.build()
    from paper_2510_26577_b200 import replicas, workloads as wl

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    rep = replicas.init("nccl")  # N > 1: independent replicas, one per GPU; no data-path collective
    rank, world = rep.rank, rep.world
    w = replicas.workload_for_rank(w, rank)
    r = measure(args, w, rep, full=True)
    if r is None or rank != 0:
        replicas.shutdown(rep)
        return

    cpu = None
    if not (args.no_cpu_baseline or args.quick):
        sec, desc, threads, ntok, _ = oracle_step_seconds(w)
        cpu = {"value": ntok / sec, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
               "ms_per_step": sec * 1e3}

    table = [table_row(r)]
    if world == 1 and not (args.no_table or args.quick or args.only):
        for name in TABLE_WORKLOADS:
            if name == w.name:
                continue
            gc.collect()
            torch.cuda.empty_cache()
            try:
                table.append(table_row(measure(args, wl.CONFIGS[name], rep, full=False)))
            except Exception as exc:  # a workload that does not fit or fails must not take the headline with it
                table.append({"workload": name, "error": f"{type(exc).__name__}: {exc}"[:200]})

    line = {
        "metric": METRIC, "value": r["total_tokens"] / (r["ms_step"] * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.kv_dtype, "data": "synthetic",
        "config": static_config(w, r["tokens_per_step"], world),
        "timing": {"l2": "distinct KV buffers per layer: the step's working set exceeds 2x L2; phases timed alone "
                         "rotate through copies of their logits (more than 2x L2) so that they read cold too",
                   "cuda_graph": True, "accept_len_mean": r["accept_mean"]},
        "e2e": r["e2e"],
        "gpu_launches": args.steps * r["launches_per_step"],
        "clocks": r["clocks"],
        "phases": r["phases"],
        "roofline": r["roofline"],
        "roofline_sweeps": r["sweeps"],
        "workloads": table,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    replicas.shutdown(rep)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_llama8b")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only", default="", choices=["", "tree", "attention", "accept", "accept_stochastic", "compact"],
                    help="profiling aid: run one phase only, without graphs")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: override the number of attention layers (smaller device footprint)")
    ap.add_argument("--no-table", action="store_true",
                    help="skip the short passes over the other configurations (the `workloads` table)")
    ap.add_argument("--quick", action="store_true",
                    help="profiling mode: few replays per phase, one end-to-end step, no CPU baseline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2510_26577_b200 import workloads as wl
    w = wl.CONFIGS[args.workload]
    if args.layers > 0:
        import dataclasses
        w = dataclasses.replace(w, n_layers=args.layers)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
