"""The classifier's target half computed inside the LM-head projection (aj_fuse_judge; the paper's
Section 3.2, "Classifier model & training": the classifier can be fused with the LM head).  The
oracle is unchanged: it evaluates sigmoid(b + w . [h_draft ; h_target]) in fp64; with the target half
taken from three extra bf16 rows of the projection the device must still agree within the tolerance
stated for judge_p, on every projection kernel, both layouts of the LM head, and every variant of
the cycle that consults the classifier."""
import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import TOL_P, DeviceCase, check_parity, check_self_consistency

pytestmark = pytest.mark.gpu


def _oracle():
    from oracle import aj_oracle as orc

    return orc


def _planted(cfg, layout=0):
    orc = _oracle()
    W = gen.make_W(cfg, layout)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype, layout)] for b in range(cfg.B)])
    return W, ht, hd, w, gen.plant_draft_tokens(cfg, y)


SHAPES = [
    # name, B, K, d, d_draft, V, flags, layout, kernel
    ("vm32", 1, 16, 1024, 512, 3000, 0, 0, "umma_vm_128x32"),
    ("vm64_many_tiles", 1, 39, 128, 64, 60000, 0, 0, "umma_vm_128x64"),     # the classifier block is one of several tiles of a CTA
    ("vm128_target_only", 4, 24, 256, 0, 2048, 0, 0, "umma_vm_128x128"),    # d_draft = 0: the judge kernel reads no features at all
    ("vm256_two_row_tiles", 5, 59, 256, 128, 5000, 8, 0, "umma_vm_128x256"),
    ("pair_narrow", 5, 39, 320, 64, 3000, 0, 0, "umma_pair_256x256"),        # M = 200
    ("pair_wide", 5, 60, 512, 256, 5000, 0, 0, "umma_pair_256x256"),         # M = 305: 160 + 160 rows on two accumulators
    ("pair_wide_two_row_tiles", 10, 59, 128, 64, 60000, 0, 0, "umma_pair_256x256"),  # M = 600, several tiles per pair
    ("vm32_dv", 1, 16, 256, 128, 3000, 0, 1, "umma_vm_128x32"),              # LM head stored [d, V]: the rows are stored [d, 8]
    ("pair_wide_dv", 5, 60, 256, 128, 5000, 0, 1, "umma_pair_256x256"),
]


@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_fused_judge_matches_the_oracle_and_the_unfused_path(shape):
    orc = _oracle()
    name, B, K, d, dd, V, flags, layout, path = shape
    cfg = gen.Config(name, B=B, K=K, d=d, d_draft=dd, V=V, sigma_W=0.2, sigma_w=0.05, match_lo=0.4, match_hi=0.9, seed=33)
    W, ht, hd, w, tok = _planted(cfg, layout)
    case = DeviceCase(cfg, W, ht, hd, w, layout=layout, flags=flags)
    try:
        plain = {tau: case.run(tok, tau) for tau in (0.0, 0.5, 1.0)}
        case.handle.fuse_judge(case.w)
        for tau in (0.0, 0.5, 1.0):
            o = orc.verify(ht, hd, W, tok, w, cfg.judge_b, tau, cfg.dtype, layout)
            g = case.run(tok, tau)
            assert g.path == path and g.launches == 2
            rep = check_parity(o, g, tok, tau)
            check_self_consistency(g, tok, tau, cfg.V)
            assert rep.max_p_err <= TOL_P
            # the projection itself is untouched by the extra block
            np.testing.assert_array_equal(g.target_tok, plain[tau].target_tok)
            np.testing.assert_array_equal(g.top1, plain[tau].top1)
            np.testing.assert_allclose(g.judge_p, plain[tau].judge_p, rtol=0, atol=2 * TOL_P, equal_nan=True)
        # a second set of weights, then back to the judge kernel: the handle follows
        w2 = (w * np.float32(-1.5)).astype(np.float32)
        import torch

        w2_d = torch.from_numpy(w2).cuda()
        case.handle.fuse_judge(w2_d)
        case.w = w2_d
        o = orc.verify(ht, hd, W, tok, w2, cfg.judge_b, 0.5, cfg.dtype, layout)
        check_parity(o, case.run(tok, 0.5), tok, 0.5)
        case.handle.fuse_judge(None)
        g = case.run(tok, 0.5)
        check_parity(o, g, tok, 0.5)
    finally:
        case.close()


def test_weights_that_need_all_three_rows():
    """Weights with 24 significant bits and a wide range of magnitudes: one bf16 row would miss the
    tolerance on p by orders of magnitude, three rows reproduce the fp32 weights exactly."""
    orc = _oracle()
    cfg = gen.Config("fold_precision", B=3, K=30, d=4096, d_draft=0, V=1500, sigma_W=0.2, sigma_w=0.02, match_lo=0.0, match_hi=0.1, seed=34)
    W, ht, hd, w, tok = _planted(cfg)
    rng = np.random.default_rng(5)
    w = (w * np.exp2(rng.integers(-6, 3, size=w.shape)).astype(np.float32) * (1 + rng.random(w.shape, dtype=np.float32) * 2.0 ** -9)).astype(np.float32)
    w *= np.float32(0.5 / np.sqrt((w.astype(np.float64) ** 2).sum()))  # keeps z of order one: p away from 0 and 1
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        case.handle.fuse_judge(case.w)
        o = orc.verify(ht, hd, W, tok, w, 0.1, 0.5, cfg.dtype)
        g = case.run(tok, 0.5, judge_b=0.1)
        rep = check_parity(o, g, tok, 0.5)
        judged = ~np.isnan(o.judge_p)
        assert judged.sum() >= 60 and rep.max_p_err <= 2e-5
        assert 0.05 < np.nanmin(o.judge_p) and np.nanmax(o.judge_p) < 0.95
    finally:
        case.close()


def test_fused_judge_with_the_variants_of_the_cycle():
    """Without the extra row, with sampled target tokens, on tree drafts, and ignored under the top-K rule."""
    import paper_2504_20039_b200 as aj

    orc = _oracle()
    cfg = gen.Config("fold_variants", B=4, K=20, d=256, d_draft=128, V=4000, sigma_W=0.2, sigma_w=0.05, match_lo=0.4, match_hi=0.9, seed=35)
    W, ht, hd, w, tok = _planted(cfg)
    # K rows per sequence: a mismatch at the last position is rejected unjudged
    case = DeviceCase(cfg, W, ht[:, : cfg.K].copy(), hd[:, : cfg.K].copy(), w, flags=aj.AJ_FLAG_NO_EXTRA_ROW)
    try:
        case.handle.fuse_judge(case.w)
        o = orc.verify(ht[:, : cfg.K], hd[:, : cfg.K], W, tok, w, cfg.judge_b, 0.5, cfg.dtype, extra_row=False)
        check_parity(o, case.run(tok, 0.5), tok, 0.5)
    finally:
        case.close()
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        case.handle.fuse_judge(case.w)
        # sampled target tokens: the noise must not touch the classifier rows
        case.handle.set_sampling(0.8, 7, 3)
        o = orc.verify(ht, hd, W, tok, w, cfg.judge_b, 0.5, cfg.dtype, temperature=0.8, seed=7, step=3)
        check_parity(o, case.run(tok, 0.5), tok, 0.5)
        case.handle.set_sampling(0.0)
        # tree drafts: every node hangs under the node two before it
        from test_gpu_tree import check_tree, run_tree

        parent = np.tile(np.array([-1, -1] + [n - 2 for n in range(2, cfg.K)], dtype=np.int32), (cfg.B, 1))
        o = orc.verify_tree(ht, hd, W, tok, parent, w, cfg.judge_b, 0.5, cfg.dtype)
        assert check_tree(orc, o, run_tree(case, tok, parent, 0.5), tok, parent, 0.5) <= cfg.B // 2  # sequences with a near-tie row
        # the top-K rule does not consult the classifier: three launches, ranks as without the fold
        case.handle.set_top_k(5)
        g = case.run(tok, 0.5)
        assert g.launches == 3
        o = orc.verify_topk(ht, W, tok, 5, cfg.dtype, band=1e-2)
        np.testing.assert_array_equal(g.target_tok, o.target_tok)
        case.handle.set_top_k(0)
        o = orc.verify(ht, hd, W, tok, w, cfg.judge_b, 0.5, cfg.dtype)
        check_parity(o, case.run(tok, 0.5), tok, 0.5)
    finally:
        case.close()


def test_fused_judge_on_vocabulary_parallel_handles():
    """Every rank of an emulated group appends the classifier block to its own shard."""
    from test_gpu_sharded import ShardedGroup

    orc = _oracle()
    cfg = gen.Config("fold_sharded", B=5, K=60, d=256, d_draft=128, V=9001, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.95, seed=36)
    W, ht, hd, w, tok = _planted(cfg)
    one = DeviceCase(cfg, W, ht, hd, w)
    grp = ShardedGroup(cfg, one, 3)
    try:
        for h in grp.handles:
            h.fuse_judge(one.w)
        one.handle.fuse_judge(one.w)
        for tau in (0.5, 0.0, 1.0):
            o = orc.verify(ht, hd, W, tok, w, cfg.judge_b, tau, cfg.dtype)
            want = one.run(tok, tau)
            check_parity(o, want, tok, tau)
            for got in grp.cycle(tok, tau):
                check_parity(o, got, tok, tau)
                np.testing.assert_array_equal(got.target_tok, want.target_tok)
                np.testing.assert_array_equal(got.judge_p, want.judge_p)  # the same three rows against the same h_target
    finally:
        grp.close()
        one.close()


def test_fused_judge_is_refused_where_there_are_no_tensor_core_rows():
    import paper_2504_20039_b200 as aj
    import torch

    w = torch.zeros(384, dtype=torch.float32, device="cuda")
    h = aj.Handle(0, 1, 4, 256, 128, 1000, aj.AJ_F32, aj.AJ_W_VD, 0)
    try:
        assert h.fuse_judge(w, check=False) == aj.AJ_ERR_UNSUPPORTED
        assert h.fuse_judge(None, check=False) == aj.AJ_OK
    finally:
        h.destroy()
