"""GPU parity at the full benchmark sizes, in the launch configuration the benchmark times.

The CPU oracle verifies every sequence of the four named workloads; their draft tokens are planted
against the oracle's own greedy tokens.  At the points of the throughput sweep it verifies whole
sequences sampled from the batch; the other sequences there get draft tokens planted against the
device's greedy tokens (never an oracle input) and are checked through properties that hold at any
size.  Set AJ_FULL_ORACLE=1 to have the oracle verify every sequence of the sweep points too.
"""
import os

import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import DeviceCase, check_parity, check_self_consistency

pytestmark = pytest.mark.gpu

_CACHE = {}


def _orc():
    from oracle import aj_oracle as orc

    return orc


def _W(cfg):
    """Host and device copies of the LM head, shared by every workload of the same model shape."""
    key = (cfg.d, cfg.V, cfg.seed)
    if key not in _CACHE:
        _CACHE.clear()  # one LM head on the device at a time
        from aj_testlib import to_device

        Wh = gen.make_W(cfg)
        _CACHE[key] = (Wh, to_device(Wh, cfg.dtype))
    return _CACHE[key]


def _sample(cfg, n):
    if os.environ.get("AJ_FULL_ORACLE") == "1" or n >= cfg.B:
        return list(range(cfg.B))
    return sorted(set(np.linspace(0, cfg.B - 1, n).astype(int).tolist()))


def _run_workload(cfg, taus, n_sample, expect_path):
    orc = _orc()
    Wh, Wd = _W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    seqs = _sample(cfg, n_sample)
    case = DeviceCase(cfg, Wd, ht, hd, w)
    try:
        # pass 1: the device's own greedy tokens, used to plant the sequences the oracle does not see
        first = case.run(gen.random_draft_tokens(cfg), 0.5)
        tok = gen.plant_draft_tokens(cfg, first.target_tok)
        # sampled sequences: greedy tokens from the oracle, draft tokens planted against them
        o_full = orc.verify(ht[seqs], hd[seqs], Wh, np.zeros((len(seqs), cfg.K), np.int32), w, cfg.judge_b, 0.5, cfg.dtype)
        tok[seqs] = gen.plant_draft_tokens(cfg, o_full.target_tok, rows=seqs)
        # one full oracle pass on the planted tokens; other thresholds replay only the accept walk
        # on the same y and p (the replay is pinned against the full pass in the CPU tests)
        o = orc.verify(ht[seqs], hd[seqs], Wh, tok[seqs], w, cfg.judge_b, taus[0], cfg.dtype)
        np.testing.assert_array_equal(o.target_tok, o_full.target_tok)
        reports = []
        for tau in taus:
            if tau != taus[0]:
                o.accept_len, o.next_tok = orc.rewalk(o.target_tok, tok[seqs], o.judge_p, tau)
            g = case.run(tok, tau)
            assert g.path == expect_path and g.launches == 2
            reports.append(check_parity(o, g, tok[seqs], tau, seqs=seqs))
            check_self_consistency(g, tok, tau, cfg.V)
        return reports
    finally:
        case.close()


def test_c2_8b_batch1_every_row():
    reps = _run_workload(gen.C2, gen.C2_TAUS, gen.C2.B, "umma_vm_128x32")
    assert all(r.rows == 17 for r in reps)


def test_c3_8b_batched_every_sequence():
    reps = _run_workload(gen.C3, (gen.C3.tau,), gen.C3.B, "umma_pair_256x256")
    assert reps[0].seqs == gen.C3.B and reps[0].rows == gen.C3.M and reps[0].seqs_exempt <= reps[0].seqs // 2


SWEEP_POINTS = [
    # B, K, kernel, (wide tiles, row tiles) of the two-SM kernel: every kernel configuration the sweep reaches
    (1, 8, "umma_vm_128x32", None),       # M = 9
    (1, 32, "umma_vm_128x64", None),      # M = 33
    (1, 64, "umma_vm_128x128", None),     # M = 65
    (8, 8, "umma_vm_128x128", None),      # M = 72
    (8, 16, "umma_pair_256x256", (0, 1)),   # M = 136: one narrow tile of 144 rows
    (8, 32, "umma_pair_256x256", (1, 1)),   # M = 264: one wide tile (144 + 128 rows), the HBM / tensor crossover
    (8, 64, "umma_pair_256x256", (1, 2)),   # M = 520: two wide tiles
    (64, 8, "umma_pair_256x256", (1, 2)),   # M = 576
    (256, 8, "umma_pair_256x256", (1, 5)),  # M = 2304
    (256, 64, "umma_pair_256x256", (1, 33)),  # M = 16640: the largest point, row tiles walked in four groups
]


@pytest.mark.parametrize("point", SWEEP_POINTS, ids=[f"b{p[0]}_k{p[1]}" for p in SWEEP_POINTS])
def test_c5_sweep_points_on_the_8b_shape(point):
    import paper_2504_20039_b200 as aj

    B, K, path, tiles = point
    cfg = gen.sweep_config(B, K)
    if tiles is not None:
        s = aj.pair_schedule(cfg.M, cfg.d, cfg.V)
        assert (s["dual"], s["n_n"]) == tiles
    reps = _run_workload(cfg, (0.5,), 3, path)
    assert reps[0].seqs >= min(B, 3)


def test_c4_70b_every_sequence_tau_sweep():
    reps = _run_workload(gen.C4, gen.C4_TAUS, gen.C4.B, "umma_pair_256x256")
    assert len(reps) == 9 and all(r.seqs == gen.C4.B and r.rows == gen.C4.M for r in reps)


def test_c2_with_the_lm_head_stored_d_by_v_gives_the_same_bits():
    """The [d, V] layout of W_lm (tensor-core path, MN-major operand) against the [V, d] layout, which the
    tests above check against the oracle: same tokens, same winning logits, at the full vocabulary."""
    cfg = gen.C2
    Wh, Wd = _W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    tok = gen.random_draft_tokens(cfg)
    a = DeviceCase(cfg, Wd, ht, hd, w, layout=0)
    b = DeviceCase(cfg, Wd.t().contiguous(), ht, hd, w, layout=1)
    try:
        ra, rb = a.run(tok, 0.5), b.run(tok, 0.5)
        assert ra.path == rb.path == "umma_vm_128x32"
        np.testing.assert_array_equal(ra.target_tok, rb.target_tok)
        np.testing.assert_array_equal(ra.top1, rb.top1)
        np.testing.assert_array_equal(ra.accept_len, rb.accept_len)
        np.testing.assert_array_equal(ra.next_tok, rb.next_tok)
    finally:
        a.close()
        b.close()


def test_c2_under_the_top_k_rule():
    """The batch-1 8B shape under the top-K rule (k = 1, 8, 1000): ranks over the full vocabulary."""
    orc = _orc()
    cfg = gen.C2
    Wh, Wd = _W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], Wh, cfg.dtype)] for b in range(cfg.B)])
    tok = gen.plant_draft_tokens(cfg, y)
    case = DeviceCase(cfg, Wd, ht, hd, w)
    try:
        for k in (1, 8, 1000):
            case.handle.set_top_k(k)
            o = orc.verify_topk(ht, Wh, tok, k, cfg.dtype, band=1e-2)
            g = case.run(tok, 0.5)
            assert g.path == "umma_vm_128x32" and g.launches == 3
            np.testing.assert_array_equal(g.target_tok, o.target_tok)
            mism = o.rank[0] >= 0
            got, want, near = g.judge_p[0][mism], o.rank[0][mism], o.near[0][mism]
            exact = want + near < k  # below top_k the rank is exact; the count of a rejected token stops at top_k or later
            assert (np.abs(got - want) <= near)[exact].all()
            assert (got[~exact] >= np.minimum(k, want - near)[~exact]).all() and (got[~exact] <= (want + near)[~exact]).all()
            n = int(o.accept_len[0])
            shaky = (mism[: n + 1] & (np.abs(o.rank[0][: n + 1] - k) <= o.near[0][: n + 1]) & (o.near[0][: n + 1] > 0)).any()
            if not shaky:
                assert g.accept_len[0] == n and g.next_tok[0] == o.next_tok[0]
    finally:
        case.close()


def test_c2_and_c3_with_sampled_target_tokens():
    """Sampled verification at the full vocabulary: every row of the batch-1 shape on the one-SM kernel, sampled
    sequences of the batched shape on the CTA-pair kernel; draft tokens planted against the oracle's own draws."""
    orc = _orc()
    for cfg, n_sample, path, T, seed, step in ((gen.C2, 1, "umma_vm_128x32", 0.7, 11, 5), (gen.C3, 3, "umma_pair_256x256", 1.0, 12, 40)):
        Wh, Wd = _W(cfg)
        ht, hd = gen.make_hidden(cfg)
        w = gen.make_judge(cfg)
        seqs = _sample(cfg, n_sample)
        R = cfg.K + 1

        def oracle(b, tok_b):  # sequence b alone, with the noise its rows have in the full batch
            return orc.verify(ht[b : b + 1], hd[b : b + 1], Wh, tok_b, w, cfg.judge_b, cfg.tau, cfg.dtype,
                              temperature=T, seed=seed, step=step, row0=b * R)

        case = DeviceCase(cfg, Wd, ht, hd, w)
        try:
            case.handle.set_sampling(T, seed, step)
            first = case.run(gen.random_draft_tokens(cfg), 0.5)       # the device's own draws, for the sequences the oracle does not see
            tok = gen.plant_draft_tokens(cfg, first.target_tok)
            for b in seqs:
                drawn = oracle(b, np.zeros((1, cfg.K), np.int32)).target_tok
                tok[b] = gen.plant_draft_tokens(cfg, drawn, rows=[b])[0]
            case.handle.set_sampling(T, seed, step)                   # the same cycle again
            g = case.run(tok, cfg.tau)
            assert g.path == path and g.launches == 2
            np.testing.assert_array_equal(g.target_tok, first.target_tok)  # same state, same draws
            for b in seqs:
                rep = check_parity(oracle(b, tok[b : b + 1]), g, tok[b : b + 1], cfg.tau, seqs=[b])
                assert rep.rows == R
            check_self_consistency(g, tok, cfg.tau, cfg.V)
            greedy = orc.verify(ht[:1], hd[:1], Wh, tok[:1], w, cfg.judge_b, cfg.tau, cfg.dtype).target_tok
            assert (greedy != g.target_tok[:1]).any()
        finally:
            case.close()


def test_c2_as_a_tree():
    """The batch-1 8B shape with its 16 draft tokens arranged as a tree (two candidates per level)."""
    orc = _orc()
    cfg = gen.C2
    Wh, Wd = _W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    N = cfg.K
    parent = np.array([[-1, -1] + [n - 2 - (n % 2) for n in range(2, N)]], dtype=np.int32)  # nodes 2l, 2l+1 hang under node 2(l-1)
    y = np.array([[orc.argmax(r)[0] for r in orc.logits(ht[0], Wh, cfg.dtype)]])
    rng = np.random.default_rng(4)
    want = y[0][parent[0] + 1]
    tok = np.where(rng.random(N) < 0.8, want, (want + 1 + rng.integers(0, cfg.V - 1, N)) % cfg.V).astype(np.int32)[None, :]
    from test_gpu_tree import check_tree, run_tree

    case = DeviceCase(cfg, Wd, ht, hd, w)
    try:
        for tau in (0.0, 0.5, 1.0):
            o = orc.verify_tree(ht, hd, Wh, tok, parent, w, cfg.judge_b, tau, cfg.dtype)
            g = run_tree(case, tok, parent, tau)
            assert case.handle.last_gemm_path() == "umma_vm_128x32"
            assert check_tree(orc, o, g, tok, parent, tau) == 0
            np.testing.assert_array_equal(g["tt"], y)
        assert g["acc"][0] == N // 2  # tau = 1: the deepest level
    finally:
        case.close()
