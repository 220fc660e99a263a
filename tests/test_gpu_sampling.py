"""Sampled verification (paper Appendix A: the target's token is drawn by the Gumbel-max trick with noise that
is a function of the random state) on the CUDA library against the CPU oracle: the same draws on every
kernel, under vocabulary sharding and from cycle to cycle, and the frequencies of the draws follow the softmax."""
import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import DeviceCase, check_parity
from test_gpu_sharded import ShardedGroup

pytestmark = pytest.mark.gpu


def _orc():
    from oracle import aj_oracle as orc

    return orc


SHAPES = [
    # name, B, K, d, d_draft, V, dtype, layout, flags, path
    ("one_sm", 3, 9, 256, 64, 3000, gen.BF16, 0, 0, "umma_vm_128x32"),
    ("one_sm_wide", 6, 20, 192, 0, 1000, gen.BF16, 0, 0, "umma_vm_128x128"),
    ("one_sm_many_rows", 9, 63, 128, 64, 2000, gen.BF16, 0, 8, "umma_vm_128x256"),
    ("pair_single", 9, 63, 128, 64, 2000, gen.BF16, 0, 0, "umma_pair_256x256"),
    ("pair_dual", 5, 60, 256, 0, 5000, gen.BF16, 0, 0, "umma_pair_256x256"),
    ("dv_layout", 5, 60, 256, 128, 5000, gen.BF16, 1, 0, "umma_pair_256x256"),
    ("dv_layout_one_sm", 2, 11, 128, 0, 1536, gen.BF16, 1, 0, "umma_vm_128x32"),
    ("cuda_cores_f32", 3, 9, 200, 40, 1234, gen.F32, 0, 0, "simt"),
    ("cuda_cores_bf16", 2, 7, 128, 0, 999, gen.BF16, 0, 1, "simt"),
    ("no_extra_row", 4, 10, 128, 64, 1024, gen.BF16, 0, 16, "umma_vm_128x64"),
]


def _inputs(name, B, K, d, dd, V, dtype, layout, seed=51):
    orc = _orc()
    cfg = gen.Config(name, B=B, K=K, d=d, d_draft=dd, V=V, dtype=dtype, sigma_W=0.2, sigma_w=0.05, match_lo=0.3, match_hi=0.8, seed=seed)
    W = gen.make_W(cfg, layout)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    return orc, cfg, W, ht, hd, w


@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_sampled_cycle_matches_the_oracle(shape):
    name, B, K, d, dd, V, dtype, layout, flags, path = shape
    orc, cfg, W, ht, hd, w = _inputs(name, B, K, d, dd, V, dtype, layout)
    extra = not (flags & 16)
    R = K + 1 if extra else K
    ht_used = ht if extra else np.ascontiguousarray(ht[:, :K])
    hd_used = hd if (extra or hd is None) else np.ascontiguousarray(hd[:, :K])
    case = DeviceCase(cfg, W, ht_used, hd_used, w, layout=layout, flags=flags)
    try:
        for T, seed, step in ((0.7, 1234, 0), (1.5, (0xFEEDFACE << 32) | 77, (5 << 32) | 3)):
            # draft tokens: the oracle's own draws at this state, with mismatches planted
            drawn = orc.verify(ht_used, hd_used, W, np.zeros((B, K), np.int32), w, cfg.judge_b, 0.0, dtype, layout, extra_row=extra,
                               temperature=T, seed=seed, step=step).target_tok
            tok = gen.plant_draft_tokens(cfg, drawn if extra else np.concatenate([drawn, drawn[:, :1]], axis=1))
            case.handle.set_sampling(T, seed, step)
            for cyc, tau in enumerate((0.5, 0.0)):  # the counter advances by one per cycle
                o = orc.verify(ht_used, hd_used, W, tok, w, cfg.judge_b, tau, dtype, layout, extra_row=extra,
                               temperature=T, seed=seed, step=step + cyc)
                g = case.run(tok, tau)
                assert g.path == path and g.launches == 2
                assert g.target_tok.shape == (B, R)
                rep = check_parity(o, g, tok, tau)
                assert rep.rows_exempt <= max(3, rep.rows // 10), rep
            if step == 0:  # a replay of the first cycle reproduces it bit for bit
                case.handle.set_sampling(T, seed, 0)
                g0 = case.run(tok, 0.5)
                case.handle.set_sampling(T, seed, 0)
                g1 = case.run(tok, 0.5)
                for a, b in ((g0.target_tok, g1.target_tok), (g0.top1, g1.top1), (g0.accept_len, g1.accept_len), (g0.judge_p, g1.judge_p)):
                    np.testing.assert_array_equal(a, b)
        # the draws differ from the greedy tokens, and temperature 0 brings greedy verification back
        greedy = orc.verify(ht_used, hd_used, W, tok, w, cfg.judge_b, 0.5, dtype, layout, extra_row=extra)
        assert (o.target_tok != greedy.target_tok).mean() > 0.2
        case.handle.set_sampling(0.0)
        g = case.run(tok, 0.5)
        assert g.launches == 2
        check_parity(greedy, g, tok, 0.5)
    finally:
        case.close()


@pytest.mark.parametrize("T", [0.02, 0.2, 6.0, 40.0])
def test_very_low_and_very_high_temperatures(T):
    """The tensor-core kernels take the logarithms only of the draws that can still take a row over; how many
    those are depends on the temperature (nearly none when it is low, nearly all when it is high, where the
    noise dwarfs the logits).  Both ends, on the one-SM kernel and on narrow and wide two-SM tiles, over several
    vocabulary tiles per CTA."""
    for name, B, K, d, dd, V, flags, path in (("t_one_sm", 2, 14, 128, 64, 40000, 0, "umma_vm_128x32"),
                                              ("t_pair_narrow", 4, 49, 128, 0, 50000, 0, "umma_pair_256x256"),
                                              ("t_pair_wide", 10, 59, 128, 64, 60000, 0, "umma_pair_256x256")):
        orc, cfg, W, ht, hd, w = _inputs(name, B, K, d, dd, V, gen.BF16, 0, seed=77)
        case = DeviceCase(cfg, W, ht, hd, w, flags=flags)
        try:
            drawn = orc.verify(ht, hd, W, np.zeros((B, K), np.int32), w, cfg.judge_b, 0.0, gen.BF16, temperature=T, seed=5, step=9).target_tok
            tok = gen.plant_draft_tokens(cfg, drawn)
            case.handle.set_sampling(T, 5, 9)
            o = orc.verify(ht, hd, W, tok, w, cfg.judge_b, 0.5, gen.BF16, temperature=T, seed=5, step=9)
            g = case.run(tok, 0.5)
            assert g.path == path
            rep = check_parity(o, g, tok, 0.5)
            assert rep.rows_exempt <= max(3, rep.rows // 10), rep
        finally:
            case.close()


def test_every_kernel_draws_the_same_tokens():
    """One input, one random state: the one-SM kernel, the CTA-pair kernel, and the CUDA-core kernel see the
    same noise, so they agree wherever the noisy scores are not too close to call."""
    orc, cfg, W, ht, hd, w = _inputs("same_noise", 5, 60, 256, 0, 4096, gen.BF16, 0)
    tok = np.zeros((cfg.B, cfg.K), np.int32)
    o = orc.verify(ht, None, W, tok, w, 0.0, 0.0, gen.BF16, temperature=1.0, seed=9, step=4)
    clear = o.gap > 1e-2
    outs = {}
    for flags in (0, 8, 1):
        case = DeviceCase(cfg, W, ht, None, w, flags=flags)
        try:
            case.handle.set_sampling(1.0, 9, 4)
            g = case.run(tok, 0.0)
            outs[g.path] = g
            assert (g.target_tok[clear] == o.target_tok[clear]).all()
        finally:
            case.close()
    assert set(outs) == {"umma_pair_256x256", "umma_vm_128x256", "simt"}
    for a in outs.values():
        np.testing.assert_allclose(a.top1, o.top1, rtol=0, atol=2e-2)
    np.testing.assert_allclose(outs["umma_pair_256x256"].top1, outs["umma_vm_128x256"].top1, rtol=0, atol=1e-4)


@pytest.mark.parametrize("world,B,K,V", [(2, 2, 7, 5000), (8, 5, 60, 9001)])
def test_vocabulary_shards_draw_what_the_unsharded_handle_draws(world, B, K, V):
    orc, cfg, W, ht, hd, w = _inputs("sharded_noise", B, K, 256, 128, V, gen.BF16, 0)
    drawn = orc.verify(ht, hd, W, np.zeros((B, K), np.int32), w, cfg.judge_b, 0.0, gen.BF16, temperature=0.9, seed=31, step=100).target_tok
    tok = gen.plant_draft_tokens(cfg, drawn)
    one = DeviceCase(cfg, W, ht, hd, w)
    grp = ShardedGroup(cfg, one, world)
    try:
        one.handle.set_sampling(0.9, 31, 100)
        for h in grp.handles:
            h.set_sampling(0.9, 31, 100)
        for cyc in range(3):
            want = one.run(tok, 0.5)
            check_parity(orc.verify(ht, hd, W, tok, w, cfg.judge_b, 0.5, gen.BF16, temperature=0.9, seed=31, step=100 + cyc), want, tok, 0.5)
            for g in grp.cycle(tok, 0.5):
                np.testing.assert_array_equal(g.target_tok, want.target_tok)
                np.testing.assert_array_equal(g.top1, want.top1)
                np.testing.assert_array_equal(g.accept_len, want.accept_len)
                np.testing.assert_array_equal(g.next_tok, want.next_tok)
    finally:
        grp.close()
        one.close()


def test_draw_frequencies_follow_the_softmax():
    """All rows carry the same hidden state, hence the same logits, but independent noise: the drawn tokens of
    many rows and cycles are a sample of softmax(logit / T) (chi-square against the oracle's logits)."""
    orc = _orc()
    from scipy.stats import chi2 as chi2_dist

    V, d, T, B, K = 256, 64, 0.8, 8, 15
    cfg = gen.Config("freq", B=B, K=K, d=d, d_draft=0, V=V, sigma_W=0.08, seed=61)
    W = gen.make_W(cfg)
    ht, _ = gen.make_hidden(cfg)
    ht[:] = ht[0, 0]
    w = gen.make_judge(cfg)
    lg = orc.logits(ht[0, :1], W, gen.BF16)[0]
    p = np.exp((lg - lg.max()) / T)
    p /= p.sum()
    cycles = 300
    n = cycles * B * (K + 1)
    assert n * p.min() >= 5 and p.max() / p.min() > 10  # every cell is populated, and the distribution is far from flat
    tok = np.zeros((B, K), np.int32)
    case = DeviceCase(cfg, W, ht, None, w)
    try:
        case.handle.set_sampling(T, 2025, 0)
        counts = np.zeros(V)
        for _ in range(cycles):
            g = case.run(tok, 0.0)
            counts += np.bincount(g.target_tok.ravel(), minlength=V)
        assert counts.sum() == n
        chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
        assert chi2 < chi2_dist.ppf(1 - 1e-4, V - 1), chi2
        # and the statistic tells the temperature: the same counts do not fit softmax(logit / (1.25 T))
        p_other = np.exp((lg - lg.max()) / (1.25 * T))
        p_other /= p_other.sum()
        assert ((counts - n * p_other) ** 2 / (n * p_other)).sum() > 2 * chi2_dist.ppf(1 - 1e-4, V - 1)
    finally:
        case.close()


def test_sampling_is_refused_where_it_is_not_defined():
    import paper_2504_20039_b200 as aj

    h = aj.Handle(0, 2, 4, 128, 0, 512)
    try:
        assert h.set_sampling(-1.0, check=False) == aj.AJ_ERR_INVALID_ARG
        assert h.set_sampling(float("nan"), check=False) == aj.AJ_ERR_INVALID_ARG
        assert h.set_sampling(float("inf"), check=False) == aj.AJ_ERR_INVALID_ARG
        h.set_top_k(4)
        assert h.set_sampling(1.0, check=False) == aj.AJ_ERR_UNSUPPORTED   # the top-K rule ranks the plain logits
        h.set_top_k(0)
        h.set_sampling(1.0, 1, 2)
        assert h.set_top_k(4, check=False) == aj.AJ_ERR_UNSUPPORTED
        h.set_sampling(0.0)
        h.set_top_k(4)
    finally:
        h.destroy()
