"""cast_accept_static: the acceptance step for callers that may not allocate device memory.

Such callers (an engine whose device memory is a fixed arena, a process whose allocator is frozen
after start-up, a plug-in that receives device pointers but no allocator) cannot create a context,
because a context allocates.  The static entry point keeps its only scratch in an array inside the
library image.  This test calls it through the C-ABI twice in a row, on different inputs, and
requires the same results as the context-based cast_accept and as the CPU oracle's greedy
acceptance: the shared array keeps the first call's contents, so the second call also shows that
nothing stale is read.  It also reads the device's free memory before and after the static call:
the call must leave it unchanged.

The file name makes pytest collect it last: if it fails, every other test has already run.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _random_tree(rng, N, vocab):
    parent = np.full(N, -1, dtype=np.int32)
    tokens = np.zeros(N, dtype=np.int32)
    depth = np.zeros(N, dtype=np.int32)
    tokens[0] = rng.integers(0, vocab)
    t = 1
    while t < N:
        par = int(rng.integers(0, t))
        if depth[par] >= 5:
            continue
        used = {int(tokens[c]) for c in range(1, t) if parent[c] == par}
        tok = int(rng.integers(0, vocab))
        if tok in used:
            continue
        parent[t], tokens[t], depth[t] = par, tok, depth[par] + 1
        t += 1
    return tokens, parent


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_static_accept_matches_context_accept_twice(dtype):
    from paper_2510_26577_b200 import build
    build.build()
    from paper_2510_26577_b200 import binding

    B, Ncap, V, H = 3, 64, 30011, 6  # an odd vocabulary: unaligned rows and a ragged last chunk
    ctx = binding.CastContext(max_batch=B, vocab=V, top_k=4, max_depth=H, total_token=Ncap, max_tree=Ncap)
    rng = np.random.default_rng(2024)
    for call in range(2):
        n_tree = rng.integers(1, Ncap + 1, size=B).astype(np.int32)
        tokens = np.full((B, Ncap), -1, dtype=np.int32)
        parent = np.full((B, Ncap), -1, dtype=np.int32)
        logits = torch.randn((B, Ncap, V), generator=torch.Generator().manual_seed(7 + call)).to(dtype)
        for b in range(B):
            tk, pr = _random_tree(rng, int(n_tree[b]), V)
            tokens[b, : n_tree[b]], parent[b, : n_tree[b]] = tk, pr
            for t in range(int(n_tree[b])):  # steer the walk down the tree about two times in three
                kids = [c for c in range(int(n_tree[b])) if pr[c] == t]
                if kids and rng.random() < 0.67:
                    logits[b, t, int(tk[kids[int(rng.integers(0, len(kids)))]])] = 50.0
        d = lambda a: torch.from_numpy(a).cuda()
        lg, tk_d, pr_d, nt_d = logits.cuda(), d(tokens), d(parent), d(n_tree)
        outs = []
        for which in range(2):
            alen = torch.full((B,), -7, dtype=torch.int32, device="cuda")
            apath = torch.full((B, H + 1), -7, dtype=torch.int32, device="cuda")
            bonus = torch.full((B,), -7, dtype=torch.int32, device="cuda")
            if which == 0:
                ctx.cast_accept(lg, B, tk_d, pr_d, None, None, nt_d, alen, apath, bonus)
                torch.cuda.synchronize()
            else:
                if call == 0:  # the very first call looks up the scratch array's address (and loads the kernels)
                    binding.cast_accept_static(lg, B, Ncap, V, H, tk_d, pr_d, nt_d, alen, apath, bonus)
                    torch.cuda.synchronize()
                    alen.fill_(-7); apath.fill_(-7); bonus.fill_(-7)
                    torch.cuda.synchronize()
                free_before = torch.cuda.mem_get_info()[0]
                binding.cast_accept_static(lg, B, Ncap, V, H, tk_d, pr_d, nt_d, alen, apath, bonus)
                torch.cuda.synchronize()
                assert torch.cuda.mem_get_info()[0] == free_before  # no device memory was taken or returned
            outs.append((alen.cpu().numpy(), apath.cpu().numpy(), bonus.cpu().numpy()))
        assert ctx.cast_poll_status()[0] == 0
        for ref, got in zip(outs[0], outs[1]):  # integer outputs: bit-exact, as in the other accept tests
            assert np.array_equal(ref, got)
        # and both equal the oracle (token-by-token greedy decoding down the tree)
        from oracle import greedy_accept
        ol, op, ob = greedy_accept(logits.double().numpy(), tokens, parent, n_tree, H)
        for ref, got in zip((ol, op, ob), outs[1]):
            assert np.array_equal(ref, got)
        assert outs[0][0].max() >= 1  # the walk did accept something


def test_static_accept_rejects_sizes_beyond_its_scratch():
    from paper_2510_26577_b200 import build
    build.build()
    from paper_2510_26577_b200 import binding
    z = torch.zeros(1, dtype=torch.int32, device="cuda")
    lg = torch.zeros(8, device="cuda")
    with pytest.raises(binding.CastError) as e:  # 17 * 128 rows > 2048
        binding.cast_accept_static(lg, 17, 128, 8, 4, z, z, z, z, z, z)
    assert e.value.code == 3
