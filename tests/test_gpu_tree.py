"""Tree drafts (paper Section 3.3 "Generality" and the EAGLE-2 appendix: the acceptance rule applied along the
root-to-leaf paths of a draft tree) on the CUDA library against the CPU oracle."""
import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import DeviceCase, GAP_EXEMPT, TOL_LOGIT, TOL_P

pytestmark = pytest.mark.gpu


def _orc():
    from oracle import aj_oracle as orc

    return orc


def make_tree(rng, N, kind):
    if kind == "chain":
        return np.arange(-1, N - 1, dtype=np.int32)
    if kind == "star":
        return np.full(N, -1, np.int32)
    if kind == "bushy":  # a few candidates per level, as a top-k expansion gives: a parent among the previous 8 nodes
        return np.array([-1 if n == 0 else int(rng.integers(max(-1, n - 8), n)) for n in range(N)], dtype=np.int32)
    return np.array([int(rng.integers(-1, n)) for n in range(N)], dtype=np.int32)  # any earlier node or the root


def plant(rng, y, parent, V, rate):
    """Draft tokens that copy the target's token of the parent's row with the given rate."""
    B, N = parent.shape
    tok = np.empty((B, N), np.int32)
    for b in range(B):
        valid = (parent[b] >= -1) & (parent[b] < np.arange(N))
        want = y[b][np.where(valid, parent[b], -1) + 1]
        other = rng.integers(0, V - 1, N)
        other = other + (other >= want)
        tok[b] = np.where(rng.random(N) < rate, want, other)
    return tok


def run_tree(case, tok, parent, tau):
    torch = case.torch
    cfg = case.cfg
    B, N = tok.shape
    i32 = dict(dtype=torch.int32, device="cuda")
    f32 = dict(dtype=torch.float32, device="cuda")
    out = dict(acc=torch.full((B,), -7, **i32), nxt=torch.full((B,), -7, **i32), best=torch.full((B,), -7, **i32),
               tt=torch.full((B, N + 1), -7, **i32), top1=torch.full((B, N + 1), 9.0, **f32), jp=torch.full((B, N), 9.0, **f32))
    tok_d = torch.from_numpy(np.ascontiguousarray(tok, dtype=np.int32)).cuda()
    par_d = torch.from_numpy(np.ascontiguousarray(parent, dtype=np.int32)).cuda()
    ht = case.ht[:B, : N + 1].contiguous()
    hd = None if case.hd is None else case.hd[:B, : N + 1].contiguous()
    case.handle.verify_tree(ht, hd, case.W, tok_d, par_d, case.w, cfg.judge_b, tau, B, N, out["acc"], out["nxt"], out["best"],
                            out["tt"], out["top1"], out["jp"], stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert case.handle.last_status() == case.aj.AJ_OK
    return {k: v.cpu().numpy() for k, v in out.items()}


def check_tree(orc, o, g, tok, parent, tau):
    """Device against oracle, plus the device against the rule applied to its own tokens and probabilities."""
    B, N = tok.shape
    exempt = 0
    for b in range(B):
        clear = o.gap[b] > GAP_EXEMPT
        assert (g["tt"][b][clear] == o.target_tok[b][clear]).all()
        assert np.abs(g["top1"][b] - o.top1[b]).max() <= TOL_LOGIT
        po, pg = o.judge_p[b], g["jp"][b].astype(np.float64)
        valid = (parent[b] >= -1) & (parent[b] < np.arange(N))
        rows_same = clear[np.where(valid, parent[b], -1) + 1]
        assert (np.isnan(po) == np.isnan(pg))[rows_same].all()
        both = ~np.isnan(po) & ~np.isnan(pg)
        assert np.abs(po[both] - pg[both]).max(initial=0.0) <= TOL_P
        assert np.isnan(pg[~valid]).all()
        near_tau = (~np.isnan(po)) & (np.abs(po - tau) <= TOL_P) & (0.0 < tau < 1.0)
        if (g["tt"][b] == o.target_tok[b]).all() and not near_tau.any():  # same tokens, no probability on the threshold: same decisions
            assert (g["acc"][b], g["best"][b], g["nxt"][b]) == (o.accept_len[b], o.best_node[b], o.next_tok[b]), b
        else:
            exempt += 1
        # whatever the rounding decided, the walk itself is exact on the device's own tokens and probabilities
        own = orc.tree_accept(tok[b], parent[b], g["tt"][b], np.nan_to_num(pg), tau)
        assert (int(g["acc"][b]), int(g["best"][b]), int(g["nxt"][b])) == own, b
    return exempt


CASES = [
    # name, B, N, d, d_draft, V, dtype, flags, tree kind, path
    ("small_random", 3, 9, 256, 128, 3000, gen.BF16, 0, "random", "umma_vm_128x32"),
    ("eagle_like", 4, 59, 256, 0, 2000, gen.BF16, 0, "bushy", "umma_pair_256x256"),
    ("wide_batch", 9, 63, 128, 64, 2000, gen.BF16, 0, "random", "umma_pair_256x256"),
    ("stars", 5, 24, 128, 64, 1000, gen.BF16, 0, "star", "umma_vm_128x128"),
    ("f32_cuda_cores", 3, 11, 72, 40, 700, gen.F32, 0, "random", "simt"),
    ("one_node", 4, 1, 64, 0, 304, gen.BF16, 0, "star", "umma_vm_128x32"),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_tree_cycle_matches_the_oracle(case):
    orc = _orc()
    name, B, N, d, dd, V, dtype, flags, kind, path = case
    cfg = gen.Config(name, B=B, K=N, d=d, d_draft=dd, V=V, dtype=dtype, sigma_W=0.2, sigma_w=0.05, seed=91)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    rng = np.random.default_rng(17)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, dtype)] for b in range(B)])
    parent = np.stack([make_tree(rng, N, kind) for _ in range(B)])
    if N > 4:
        parent[0, 3] = N + 5      # not a node
        parent[B - 1, 2] = 2      # its own parent
        parent[B - 1, 4] = -3
    tok = plant(rng, y, parent, V, 0.75)
    tok[0, 0] = -1 if N > 1 else tok[0, 0]  # an id outside the vocabulary simply never matches
    dev = DeviceCase(cfg, W, ht, hd, w, flags=flags)
    try:
        exempt = 0
        for tau in (0.5, 0.0, 1.0, 0.35):
            o = orc.verify_tree(ht, hd, W, tok, parent, w, cfg.judge_b, tau, dtype)
            g = run_tree(dev, tok, parent, tau)
            assert dev.handle.last_gemm_path() == path and dev.handle.last_launch_count() == 2
            exempt += check_tree(orc, o, g, tok, parent, tau)
            if tau >= 1.0:  # everything with a valid ancestry is accepted: the deepest node of the tree
                for b in range(B):
                    depth = np.zeros(N, int)
                    ok = np.zeros(N, bool)
                    for n in range(N):
                        q = parent[b, n]
                        if -1 <= q < n and (q == -1 or ok[q]):
                            ok[n], depth[n] = True, (0 if q == -1 else depth[q]) + 1
                    assert g["acc"][b] == depth.max() and g["best"][b] == int(np.argmax(np.where(ok, depth, -1)))
        assert exempt <= 2
        # a window is a chain: the tree entry point then returns what aj_verify returns, bit for bit
        chain = np.tile(make_tree(rng, N, "chain"), (B, 1))
        tokc = gen.plant_draft_tokens(cfg, y)
        gt = run_tree(dev, tokc, chain, 0.5)
        gw = dev.run(tokc, 0.5)
        np.testing.assert_array_equal(gt["acc"], gw.accept_len)
        np.testing.assert_array_equal(gt["nxt"], gw.next_tok)
        np.testing.assert_array_equal(gt["best"], gw.accept_len - 1)
        np.testing.assert_array_equal(gt["tt"], gw.target_tok)
        np.testing.assert_array_equal(gt["jp"], gw.judge_p)
        np.testing.assert_array_equal(gt["top1"], gw.top1)
    finally:
        dev.close()


def test_tree_cycle_with_sampled_target_tokens():
    orc = _orc()
    B, N, V = 4, 30, 1500
    cfg = gen.Config("tree_sampled", B=B, K=N, d=128, d_draft=64, V=V, sigma_W=0.2, sigma_w=0.05, seed=93)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    rng = np.random.default_rng(3)
    parent = np.stack([make_tree(rng, N, "bushy") for _ in range(B)])
    drawn = orc.verify_tree(ht, hd, W, np.zeros((B, N), np.int32), parent, w, cfg.judge_b, 0.0, gen.BF16, temperature=0.8, seed=5, step=9).target_tok
    tok = plant(rng, drawn, parent, V, 0.75)
    dev = DeviceCase(cfg, W, ht, hd, w)
    try:
        dev.handle.set_sampling(0.8, 5, 9)
        o = orc.verify_tree(ht, hd, W, tok, parent, w, cfg.judge_b, 0.5, gen.BF16, temperature=0.8, seed=5, step=9)
        g = run_tree(dev, tok, parent, 0.5)
        assert check_tree(orc, o, g, tok, parent, 0.5) <= 2
        assert o.accept_len.max() >= 2
    finally:
        dev.close()


def test_tree_entry_point_refuses_what_it_does_not_define():
    import torch

    import paper_2504_20039_b200 as aj

    def call(h, parent_ok=True):
        i32 = dict(dtype=torch.int32, device="cuda")
        ht = torch.zeros((2, 5, 128), dtype=torch.bfloat16, device="cuda")
        W = torch.zeros((512, 128), dtype=torch.bfloat16, device="cuda")
        w = torch.zeros(128, dtype=torch.float32, device="cuda")
        tok = torch.zeros((2, 4), **i32)
        par = torch.full((2, 4), -1, **i32)
        acc, nxt = torch.zeros(2, **i32), torch.zeros(2, **i32)
        st = h.verify_tree(ht, None, W, tok, par if parent_ok else None, w, 0.0, 0.5, 2, 4, acc, nxt, check=False)
        torch.cuda.synchronize()
        return st

    h = aj.Handle(0, 2, 4, 128, 0, 512)
    try:
        assert call(h) == aj.AJ_OK
        assert call(h, parent_ok=False) == aj.AJ_ERR_INVALID_ARG
        h.set_top_k(3)
        assert call(h) == aj.AJ_ERR_UNSUPPORTED
    finally:
        h.destroy()
    h = aj.Handle(0, 2, 4, 128, 0, 512, flags=aj.AJ_FLAG_NO_EXTRA_ROW)
    try:
        assert call(h) == aj.AJ_ERR_UNSUPPORTED
    finally:
        h.destroy()


def test_tree_cycle_on_a_vocabulary_parallel_handle():
    """A group of one rank: the tree entry point publishes to and gathers from its own exchange buffer and
    returns what the unsharded handle returns."""
    import torch

    import paper_2504_20039_b200 as aj

    orc = _orc()
    B, N, V = 3, 12, 2048
    cfg = gen.Config("tree_sharded", B=B, K=N, d=128, d_draft=64, V=V, sigma_W=0.2, sigma_w=0.05, seed=95)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    rng = np.random.default_rng(8)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, gen.BF16)] for b in range(B)])
    parent = np.stack([make_tree(rng, N, "random") for _ in range(B)])
    tok = plant(rng, y, parent, V, 0.7)
    dev = DeviceCase(cfg, W, ht, hd, w)
    buf = torch.zeros(aj.shard_exchange_bytes(B, N, 1) // 8, dtype=torch.int64, device="cuda")
    sharded = aj.Handle(0, B, N, cfg.d, cfg.d_draft, V, gen.BF16, aj.AJ_W_VD, 0, shard=(0, 1, 0, V, [buf]))
    try:
        want = run_tree(dev, tok, parent, 0.5)
        check_tree(orc, orc.verify_tree(ht, hd, W, tok, parent, w, cfg.judge_b, 0.5, gen.BF16), want, tok, parent, 0.5)
        plain = dev.handle
        dev.handle = sharded
        for _ in range(2):  # two cycles: both slot parities
            got = run_tree(dev, tok, parent, 0.5)
            for k in want:
                np.testing.assert_array_equal(got[k], want[k])
        dev.handle = plain
    finally:
        sharded.destroy()
        dev.close()
