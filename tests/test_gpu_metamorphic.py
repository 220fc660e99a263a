"""Properties of the verify-and-judge step that hold without an oracle, checked on the CUDA library:
relabelling the vocabulary relabels the tokens, exact scalings keep them, sequences do not see each other,
and nothing after the accepted prefix (plus the rows the judge reads there) can matter."""
import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import DeviceCase

pytestmark = pytest.mark.gpu


def _case(M_kind):
    # small: one-SM kernel; pair: two-SM kernel (M = 305)
    B, K = (3, 9) if M_kind == "small" else (5, 60)
    return gen.Config(f"meta_{M_kind}", B=B, K=K, d=256, d_draft=128, V=3001, sigma_W=0.2, sigma_w=0.05,
                      match_lo=0.5, match_hi=0.9, seed=33)


def _run(cfg, W, ht, hd, w, tok, tau=0.5):
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        return case.run(tok, tau)
    finally:
        case.close()


@pytest.mark.parametrize("kind", ["small", "pair"])
def test_permuting_the_vocabulary_permutes_the_tokens(kind):
    cfg = _case(kind)
    W, (ht, hd), w = gen.make_W(cfg), gen.make_hidden(cfg), gen.make_judge(cfg)
    base = _run(cfg, W, ht, hd, w, gen.random_draft_tokens(cfg))
    tok = gen.plant_draft_tokens(cfg, base.target_tok)
    base = _run(cfg, W, ht, hd, w, tok)
    perm = np.random.default_rng(1).permutation(cfg.V)          # new index i holds old entry perm[i]
    inv = np.argsort(perm)
    got = _run(cfg, np.ascontiguousarray(W[perm]), ht, hd, w, inv[tok].astype(np.int32))
    np.testing.assert_array_equal(got.target_tok, inv[base.target_tok])  # gaps are wide at sigma_W = 0.2: no ties to reorder
    np.testing.assert_array_equal(got.accept_len, base.accept_len)
    np.testing.assert_array_equal(got.next_tok, inv[base.next_tok])
    np.testing.assert_array_equal(got.top1, base.top1)                    # the same dot products, bit for bit
    np.testing.assert_array_equal(got.judge_p, base.judge_p)


@pytest.mark.parametrize("kind", ["small", "pair"])
def test_doubling_the_lm_head_doubles_the_logits_and_keeps_every_decision(kind):
    cfg = _case(kind)
    W, (ht, hd), w = gen.make_W(cfg), gen.make_hidden(cfg), gen.make_judge(cfg)
    base = _run(cfg, W, ht, hd, w, gen.random_draft_tokens(cfg))
    tok = gen.plant_draft_tokens(cfg, base.target_tok)
    base = _run(cfg, W, ht, hd, w, tok)
    W2 = gen.f32_to_bf16_bits(gen.bf16_bits_to_f32(W) * 2.0)              # exact in bf16
    got = _run(cfg, W2, ht, hd, w, tok)
    np.testing.assert_array_equal(got.target_tok, base.target_tok)
    np.testing.assert_array_equal(got.top1, 2.0 * base.top1)              # powers of two commute with rounding
    np.testing.assert_array_equal(got.accept_len, base.accept_len)        # the judge does not see W_lm
    np.testing.assert_array_equal(got.judge_p, base.judge_p)


@pytest.mark.parametrize("kind", ["small", "pair"])
def test_shuffling_the_batch_shuffles_the_outputs(kind):
    cfg = _case(kind)
    W, (ht, hd), w = gen.make_W(cfg), gen.make_hidden(cfg), gen.make_judge(cfg)
    base = _run(cfg, W, ht, hd, w, gen.random_draft_tokens(cfg))
    tok = gen.plant_draft_tokens(cfg, base.target_tok)
    base = _run(cfg, W, ht, hd, w, tok)
    order = np.random.default_rng(2).permutation(cfg.B)
    got = _run(cfg, W, np.ascontiguousarray(ht[order]), np.ascontiguousarray(hd[order]), w, np.ascontiguousarray(tok[order]))
    for name in ("accept_len", "next_tok", "target_tok", "top1"):
        np.testing.assert_array_equal(getattr(got, name), getattr(base, name)[order])
    np.testing.assert_array_equal(got.judge_p, base.judge_p[order])


@pytest.mark.parametrize("kind", ["small", "pair"])
def test_nothing_behind_the_stop_can_change_the_result(kind):
    cfg = _case(kind)
    W, (ht, hd), w = gen.make_W(cfg), gen.make_hidden(cfg), gen.make_judge(cfg)
    base = _run(cfg, W, ht, hd, w, gen.random_draft_tokens(cfg))
    tok = gen.plant_draft_tokens(cfg, base.target_tok)
    base = _run(cfg, W, ht, hd, w, tok)
    assert (base.accept_len < cfg.K - 2).any()  # some sequence really stops early
    ht2, hd2, tok2 = ht.copy(), hd.copy(), tok.copy()
    junk = np.random.default_rng(3)
    for b in range(cfg.B):
        n = int(base.accept_len[b])
        # position n is where the walk stops: its token, and rows up to n + 1 (which the judge reads for
        # position n), are the last things that matter
        tok2[b, n + 1 :] = junk.integers(0, cfg.V, size=cfg.K - n - 1 if n < cfg.K else 0)
        if n + 2 <= cfg.K:
            ht2[b, n + 2 :] = gen.f32_to_bf16_bits(junk.standard_normal((cfg.K - n - 1, cfg.d)).astype(np.float32))
            hd2[b, n + 2 :] = gen.f32_to_bf16_bits(junk.standard_normal((cfg.K - n - 1, cfg.d_draft)).astype(np.float32))
    got = _run(cfg, W, ht2, hd2, w, tok2)
    np.testing.assert_array_equal(got.accept_len, base.accept_len)
    np.testing.assert_array_equal(got.next_tok, base.next_tok)
