"""Pins for the CPU oracle: each test ties it to something other than itself.

- a library routine on the special case where the step *is* that routine (fp64 matmul,
  first-occurrence argmax);
- closed forms (one-hot rows turn the projection into a table lookup; unit judge weights
  turn the classifier into sigmoid(b + one feature));
- what the paper fixes about the acceptance rule (Section 2: the first mismatch and
  everything after it are rejected; Section 3.3: the classifier is consulted only where
  the original rule would reject, a forgiven token is accepted and later tokens are then
  tested as before; Section 4.3 tables: a larger threshold accepts more);
- brute force over every match / forgiven / important pattern of a short window;
- the closed-form expectation of the accepted length under the synthetic generator.
"""
import itertools
import math

import numpy as np
import pytest

import aj_inputs as gen
from oracle import aj_oracle as orc

BF16, F32 = gen.BF16, gen.F32


def _store(x, dtype):
    x = np.asarray(x, dtype=np.float32)
    return gen.f32_to_bf16_bits(x) if dtype == BF16 else x


# ---------------------------------------------------------------- projection + argmax


@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("R,d,V", [(1, 8, 5), (5, 96, 333), (17, 256, 1000), (33, 512, 4099)])
def test_logits_equal_library_matmul(dtype, layout, R, d, V):
    g = np.random.default_rng(R * 1000 + d + V)
    h = _store(g.standard_normal((R, d)), dtype)
    W = _store(g.standard_normal((V, d)) * 0.02, dtype)
    Wl = W if layout == 0 else np.ascontiguousarray(W.T)
    got = orc.logits(h, Wl, dtype, layout)
    want = gen.to_f64(h, dtype) @ gen.to_f64(W, dtype).T
    assert got.shape == (R, V)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-11)
    for r in range(R):
        y, top1, gap = orc.argmax(got[r])
        assert y == int(np.argmax(want[r]))
        assert top1 == got[r, y]
        srt = np.sort(got[r])
        assert gap == pytest.approx(srt[-1] - srt[-2], abs=1e-15)


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_one_hot_rows_read_a_column_of_W(dtype):
    # h = e_k makes logit[v] = W[k, v] exactly, so y is a lookup in W.  A transposed
    # operand or a wrong row/column index breaks this on a non-square W.
    g = np.random.default_rng(7)
    d, V = 48, 301
    Wf = g.standard_normal((V, d)).astype(np.float32)
    W = _store(Wf, dtype)
    Wv = gen.to_f64(W, dtype)
    ks = [0, 1, 17, d - 1]
    h = np.zeros((len(ks), d), np.float32)
    for r, k in enumerate(ks):
        h[r, k] = 1.0
    lg = orc.logits(_store(h, dtype), W, dtype, 0)
    for r, k in enumerate(ks):
        np.testing.assert_array_equal(lg[r], Wv[:, k])
        assert orc.argmax(lg[r])[0] == int(np.argmax(Wv[:, k]))


def test_argmax_ties_take_the_lowest_index_and_signed_zeros_tie():
    assert orc.argmax(np.array([1.0, 3.0, 3.0, 2.0]))[0] == 1
    assert orc.argmax(np.array([1.0, 3.0, 3.0, 2.0]))[2] == 0.0
    assert orc.argmax(np.array([-0.0, 0.0, -1.0]))[0] == 0
    assert orc.argmax(np.array([0.0, -0.0, -1.0]))[0] == 0
    assert orc.argmax(np.array([-5.0, -2.0, -3.0])) == (1, -2.0, 1.0)
    assert orc.argmax(np.array([4.0]))[0] == 0


def test_projection_invariants():
    g = np.random.default_rng(11)
    R, d, V = 6, 64, 257
    h = _store(g.standard_normal((R, d)), BF16)
    W = _store(g.standard_normal((V, d)) * 0.02, BF16)
    base = orc.logits(h, W, BF16)
    y0 = [orc.argmax(r)[0] for r in base]
    # permuting vocabulary entries permutes the winner
    perm = g.permutation(V)
    lp = orc.logits(h, np.ascontiguousarray(W[perm]), BF16)
    inv = np.argsort(perm)
    assert [orc.argmax(r)[0] for r in lp] == [int(inv[y]) for y in y0]
    # doubling h (exact in bf16) doubles every logit and keeps the winner
    h2 = _store(gen.bf16_bits_to_f32(h) * 2.0, BF16)
    l2 = orc.logits(h2, W, BF16)
    np.testing.assert_array_equal(l2, 2.0 * base)
    # a duplicated winning column: the lower index is returned
    for r in range(R):
        Wd = W.copy()
        hi = (y0[r] + 40) % V
        lo_i, hi_i = min(y0[r], hi), max(y0[r], hi)
        Wd[lo_i] = W[y0[r]]
        Wd[hi_i] = W[y0[r]]
        assert orc.argmax(orc.logits(h[r : r + 1], Wd, BF16)[0])[0] == lo_i


# ------------------------------------------------------------------------------- judge


def _sigmoid(z):
    return 1.0 / (1.0 + math.exp(-z))


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_judge_closed_forms(dtype):
    g = np.random.default_rng(3)
    d, dd = 40, 24
    ht = _store(g.standard_normal(d), dtype)
    hd = _store(g.standard_normal(dd), dtype)
    xt, xd = gen.to_f64(ht, dtype), gen.to_f64(hd, dtype)
    w0 = np.zeros(d + dd, np.float32)
    for b in (-2.0, 0.0, 0.75):
        assert orc.judge_p(hd, ht, dtype, w0, b) == pytest.approx(_sigmoid(b), abs=1e-15)
    # unit weight on feature f: the first d_draft features are the draft model's, then the target's
    for f in (0, 5, dd - 1, dd, dd + 7, dd + d - 1):
        w = w0.copy()
        w[f] = 1.0
        x = xd[f] if f < dd else xt[f - dd]
        assert orc.judge_p(hd, ht, dtype, w, 0.25) == pytest.approx(_sigmoid(0.25 + x), abs=1e-15)
    # general weights against a float64 dot product; p(z) + p(-z) = 1
    w = (g.standard_normal(d + dd) * 0.05).astype(np.float32)
    z = float(w[:dd].astype(np.float64) @ xd + w[dd:].astype(np.float64) @ xt)
    p = orc.judge_p(hd, ht, dtype, w, 0.0)
    assert p == pytest.approx(_sigmoid(z), abs=1e-14)
    assert p + orc.judge_p(hd, ht, dtype, -w, 0.0) == pytest.approx(1.0, abs=1e-14)
    # target-only features
    assert orc.judge_p(None, ht, dtype, w[dd:], 0.125) == pytest.approx(
        _sigmoid(0.125 + float(w[dd:].astype(np.float64) @ xt)), abs=1e-14
    )


# ---------------------------------------------------------- acceptance rule: brute force


def _controlled_case(pattern, V=9, d=9, dd=4):
    """A window whose outcome at each position is chosen by hand.

    pattern[i] in {"m", "f", "i"}: draft token matches / mismatches and is forgiven /
    mismatches and is important.  W is the identity (V = d), rows of h_target are one-hot,
    so y[j] is the position of the one; the judge reads draft feature 0 of row i+1.
    """
    K = len(pattern)
    g = np.random.default_rng(sum(3**i * "mfi".index(c) for i, c in enumerate(pattern)) + 100 * K)
    y = g.integers(0, V, size=K + 1)
    ht = np.zeros((1, K + 1, d), np.float32)
    for j in range(K + 1):
        ht[0, j, y[j]] = 1.0
    hd = np.zeros((1, K + 1, dd), np.float32)
    tok = np.empty((1, K), np.int32)
    for i, c in enumerate(pattern):
        tok[0, i] = y[i] if c == "m" else (y[i] + 1 + g.integers(0, V - 1)) % V
        hd[0, i + 1, 0] = {"m": 0.0, "f": -20.0, "i": 20.0}[c]
    hd[0, 0, 0] = 20.0  # row 0 must never be read by the judge
    w = np.zeros(dd + d, np.float32)
    w[0] = 1.0
    W = np.eye(V, d, dtype=np.float32)
    return ht, hd, W, tok, w, y


def _second_evaluator(passes):
    """Largest n such that every position before n passes (no early exit)."""
    K = len(passes)
    return max(n for n in range(K + 1) if all(passes[:n]))


@pytest.mark.parametrize("K", [1, 2, 3, 4])
def test_every_pattern_of_a_short_window(K):
    for pattern in itertools.product("mfi", repeat=K):
        ht, hd, W, tok, w, y = _controlled_case(pattern)
        r = orc.verify(ht, hd, W, tok, w, 0.0, 0.5, F32)
        want = _second_evaluator([c != "i" for c in pattern])
        assert r.accept_len[0] == want, pattern
        assert r.next_tok[0] == y[want], pattern
        np.testing.assert_array_equal(r.target_tok[0], y)
        for i, c in enumerate(pattern):
            if c == "m":
                assert math.isnan(r.judge_p[0, i])
            else:
                assert r.judge_p[0, i] == pytest.approx(_sigmoid(20.0 if c == "i" else -20.0), abs=1e-12)
        # never forgiving: plain greedy speculative decoding, stop at the first mismatch
        r0 = orc.verify(ht, hd, W, tok, w, 0.0, 0.0, F32)
        assert r0.accept_len[0] == _second_evaluator([c == "m" for c in pattern])
        # always forgiving: the whole window and the bonus token
        r1 = orc.verify(ht, hd, W, tok, w, 0.0, 1.0, F32)
        assert r1.accept_len[0] == K and r1.next_tok[0] == y[K]


@pytest.mark.parametrize("block", ["draft", "target"])
def test_judge_reads_the_row_that_encodes_the_draft_token(block):
    # one mismatch at position i; only row i+1 carries a large "important" feature, every
    # other row would forgive.  Reading row i (the state that predicted the token) instead
    # would accept.  The feature sits either in the draft block or in the target block
    # (the last target feature has a zero row in W, so it does not disturb the argmax).
    K, V, d, dd = 5, 7, 8, 3
    W = np.eye(V, d, dtype=np.float32)
    for i in range(K):
        ht = np.zeros((1, K + 1, d), np.float32)
        y = [(3 * j + 1) % V for j in range(K + 1)]
        for j in range(K + 1):
            ht[0, j, y[j]] = 1.0
        hd = np.full((1, K + 1, dd), -1.0, np.float32)
        ht[0, :, d - 1] = -1.0
        feat = (hd, 2, 2) if block == "draft" else (ht, d - 1, dd + d - 1)
        feat[0][0, i + 1, feat[1]] = 30.0
        tok = np.array([y[:K]], np.int32)
        tok[0, i] = (y[i] + 1) % V
        w = np.zeros(dd + d, np.float32)
        w[feat[2]] = 1.0
        r = orc.verify(ht, hd, W, tok, w, 0.0, 0.5, F32)
        np.testing.assert_array_equal(r.target_tok[0], y)
        assert r.accept_len[0] == i and r.next_tok[0] == y[i]
        feat[0][0, i + 1, feat[1]] = -30.0
        r = orc.verify(ht, hd, W, tok, w, 0.0, 0.5, F32)
        assert r.accept_len[0] == K


# --------------------------------------------- acceptance rule: what the paper fixes


def _random_case(cfg):
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(cfg.B)])
    tok = gen.plant_draft_tokens(cfg, y)
    return W, ht, hd, w, y, tok


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_threshold_extremes_monotonicity_and_vanilla_bound(dtype):
    cfg = gen.Config("t", B=40, K=12, d=64, d_draft=32, V=211, dtype=dtype, sigma_w=0.2, match_lo=0.4, match_hi=0.9, seed=5)
    W, ht, hd, w, y, tok = _random_case(cfg)
    mism = tok != y[:, : cfg.K]
    vanilla = np.array([int(np.argmax(np.append(m, True))) for m in mism])
    prev = None
    for tau in (0.0, 0.05, 0.2, 0.5, 0.8, 0.95, 1.0):
        r = orc.verify(ht, hd, W, tok, w, cfg.judge_b, tau, dtype)
        np.testing.assert_array_equal(r.target_tok, y)
        assert (r.accept_len >= vanilla).all()
        assert (r.next_tok == y[np.arange(cfg.B), r.accept_len]).all()
        assert (np.isnan(r.judge_p) == ~mism).all()
        if tau == 0.0:
            np.testing.assert_array_equal(r.accept_len, vanilla)
        if tau == 1.0:
            assert (r.accept_len == cfg.K).all()
        if prev is not None:
            assert (r.accept_len >= prev).all()
        prev = r.accept_len
        # the replay helper agrees with the full evaluation
        a2, n2 = orc.rewalk(r.target_tok, tok, r.judge_p, tau)
        np.testing.assert_array_equal(a2, r.accept_len)
        np.testing.assert_array_equal(n2, r.next_tok)
    assert 0 < vanilla.mean() < cfg.K  # the case is not degenerate


def test_sequences_are_independent_and_the_rejected_tail_is_never_consulted():
    cfg = gen.Config("t", B=9, K=10, d=32, d_draft=16, V=97, dtype=BF16, sigma_w=0.3, match_lo=0.5, match_hi=0.9, seed=9)
    W, ht, hd, w, y, tok = _random_case(cfg)
    full = orc.verify(ht, hd, W, tok, w, 0.0, 0.5, BF16)
    order = np.random.default_rng(0).permutation(cfg.B)
    shuf = orc.verify(ht[order], hd[order], W, tok[order], w, 0.0, 0.5, BF16)
    np.testing.assert_array_equal(shuf.accept_len, full.accept_len[order])
    np.testing.assert_array_equal(shuf.next_tok, full.next_tok[order])
    for b in range(cfg.B):
        one = orc.verify(ht[b : b + 1], hd[b : b + 1], W, tok[b : b + 1], w, 0.0, 0.5, BF16)
        assert one.accept_len[0] == full.accept_len[b] and one.next_tok[0] == full.next_tok[b]
        n = int(full.accept_len[b])
        if n + 2 <= cfg.K:  # junk after the stop changes nothing
            t2, h2, g2 = tok.copy(), ht.copy(), hd.copy()
            t2[b, n + 1 :] = 0
            h2[b, n + 2 :] = gen.f32_to_bf16_bits(np.full((cfg.K - n - 1, cfg.d), 3.0, np.float32))
            g2[b, n + 2 :] = 0
            j = orc.verify(h2[b : b + 1], g2[b : b + 1], W, t2[b : b + 1], w, 0.0, 0.5, BF16)
            assert j.accept_len[0] == n and j.next_tok[0] == full.next_tok[b]


# ------------------------------------------ generator + oracle against a closed form


def _phi(x):
    return 0.5 * (1.0 + math.erf(x / math.sqrt(2.0)))


@pytest.mark.parametrize("tau", [0.5, 0.7])
def test_expected_accept_len_matches_closed_form(tau):
    # With i.i.d. unit-variance features z ~ N(b, sigma_w^2 F), so a mismatch is forgiven
    # with probability Phi(logit(tau) / sigma_z); a position passes with q = r + (1-r) * that,
    # and E[accept_len] = sum_{i=1..K} q^i.
    r_match, K = 0.6, 8
    cfg = gen.Config("t", B=6000, K=K, d=48, d_draft=16, V=61, dtype=F32, sigma_w=0.1, match_lo=r_match, match_hi=r_match, seed=21)
    W, ht, hd, w, y, tok = _random_case(cfg)
    r = orc.verify(ht, hd, W, tok, w, 0.0, tau, F32)
    sigma_z = float(np.sqrt((w.astype(np.float64) ** 2).sum()))
    q = r_match + (1 - r_match) * _phi(math.log(tau / (1 - tau)) / sigma_z)
    want = sum(q**i for i in range(1, K + 1))
    var = sum((2 * i - 1) * q**i for i in range(1, K + 1)) - want**2  # E[N^2] - E[N]^2
    se = math.sqrt(var / cfg.B)
    assert abs(float(r.accept_len.mean()) - want) < 4 * se
    assert abs(float((tok == y[:, :K]).mean()) - r_match) < 4 * math.sqrt(r_match * (1 - r_match) / (cfg.B * K))


# ---------------------------------------------------- variant: the last draft token is not encoded


@pytest.mark.parametrize("tau", [0.0, 0.4, 1.0])
def test_without_the_extra_row_the_last_mismatch_is_rejected_unjudged(tau):
    """Section 3.2, design choice 1, second way: with K rows instead of K + 1 the states that encode the
    last draft token do not exist, so a mismatch there is discarded without the classifier.  Everything
    before the last position must be decided exactly as with the extra row."""
    g = np.random.default_rng(101)
    B, K, d, dd, V = 40, 5, 32, 16, 50
    cfg = gen.Config("noextra", B=B, K=K, d=d, d_draft=dd, V=V, sigma_W=0.3, sigma_w=0.3, match_lo=0.6, match_hi=0.9, seed=77)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(B)])
    tok = gen.plant_draft_tokens(cfg, y)
    tok[:8, K - 1] = y[:8, K - 1]                    # some sequences surely match at the last position
    tok[8:16, K - 1] = (y[8:16, K - 1] + 1) % V      # and some surely do not
    full = orc.verify(ht, hd, W, tok, w, 0.0, tau, cfg.dtype)
    ne = orc.verify(ht[:, :K].copy(), hd[:, :K].copy(), W, tok, w, 0.0, tau, cfg.dtype, extra_row=False)
    assert ne.target_tok.shape == (B, K)
    np.testing.assert_array_equal(ne.target_tok, full.target_tok[:, :K])
    np.testing.assert_array_equal(ne.top1, full.top1[:, :K])
    np.testing.assert_array_equal(ne.judge_p[:, : K - 1], full.judge_p[:, : K - 1])  # same rows, same values
    assert np.isnan(ne.judge_p[:, K - 1]).all()     # never judged at the last position
    seen = set()
    for b in range(B):
        last_mismatch = tok[b, K - 1] != y[b, K - 1]
        if full.accept_len[b] < K - 1:               # stopped earlier: nothing changes
            want_len, want_next, kind = full.accept_len[b], full.next_tok[b], "early"
        elif last_mismatch:                          # reached the last position and it mismatches
            want_len, want_next, kind = K - 1, y[b, K - 1], "last_rejected"
        else:                                        # reached it and it matches: all K pass, nothing to predict from
            want_len, want_next, kind = K, -1, "all_pass"
        seen.add(kind)
        assert (ne.accept_len[b], ne.next_tok[b]) == (want_len, want_next), (b, kind)
    assert "last_rejected" in seen and "all_pass" in seen and ("early" in seen or tau >= 1.0)


def test_without_the_extra_row_single_token_window():
    # K = 1: one row per sequence; the only position is the last one
    cfg = gen.Config("noextra1", B=6, K=1, d=16, d_draft=0, V=9, sigma_W=0.5, seed=5)
    W = gen.make_W(cfg)
    ht, _ = gen.make_hidden(cfg)
    ht = ht[:, :1].copy()
    w = gen.make_judge(cfg)
    y = np.array([orc.argmax(orc.logits(ht[b], W, cfg.dtype)[0])[0] for b in range(cfg.B)])
    tok = y.copy().reshape(-1, 1).astype(np.int32)
    tok[::2, 0] = (tok[::2, 0] + 1) % cfg.V
    r = orc.verify(ht, None, W, tok, w, 0.0, 1.0, cfg.dtype, extra_row=False)
    np.testing.assert_array_equal(r.accept_len, np.where(np.arange(cfg.B) % 2 == 0, 0, 1))
    np.testing.assert_array_equal(r.next_tok, np.where(np.arange(cfg.B) % 2 == 0, y, -1))


# ------------------------------------------------------------------- the top-K rule (Section 4.1)


def test_rank_equals_position_in_a_stable_sort():
    g = np.random.default_rng(5)
    row = np.round(g.standard_normal(300), 1)            # rounded: plenty of exact ties
    order = np.argsort(-row, kind="stable")              # decreasing logit, ties by increasing index
    pos = np.empty_like(order)
    pos[order] = np.arange(row.size)
    for tok in (0, 7, 150, 299, int(order[0]), int(order[-1])):
        r, near = orc.rank(row, tok, band=0.05)
        assert r == pos[tok]
        assert near == int((np.abs(row - row[tok]) <= 0.05).sum()) - 1
    assert orc.rank(row, int(order[0]))[0] == 0


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_top_k_rule_extremes_monotonicity_and_brute_force(dtype):
    B, K, d, V = 12, 6, 32, 40
    cfg = gen.Config("topk", B=B, K=K, d=d, d_draft=0, V=V, dtype=dtype, sigma_W=0.3, match_lo=0.3, match_hi=0.7, seed=61)
    W = gen.make_W(cfg)
    ht, _ = gen.make_hidden(cfg)
    lg = np.stack([orc.logits(ht[b], W, dtype) for b in range(B)])      # [B, K+1, V]
    y = np.stack([[orc.argmax(r)[0] for r in lg[b]] for b in range(B)])
    tok = gen.plant_draft_tokens(cfg, y)
    tok[0, 2] = -3                                                        # outside the vocabulary: never accepted
    tok[1, 1] = V + 5
    vanilla = np.array([int(np.argmax(np.append(tok[b] != y[b, :K], True))) for b in range(B)])
    prev = None
    for k in (1, 2, 3, 5, 10, V, V + 7):
        r = orc.verify_topk(ht, W, tok, k, dtype)
        np.testing.assert_array_equal(r.target_tok, y)
        # brute force from a full sort of every row
        for b in range(B):
            n = 0
            while n < K:
                t = tok[b, n]
                if t != y[b, n]:
                    if not (0 <= t < V):
                        break
                    order = np.argsort(-lg[b, n], kind="stable")
                    if int(np.nonzero(order == t)[0][0]) >= k:
                        break
                n += 1
            assert r.accept_len[b] == n and r.next_tok[b] == y[b, n]
        if k == 1:  # only the argmax itself is in the top 1, and a mismatch is not the argmax: plain greedy verification
            np.testing.assert_array_equal(r.accept_len, vanilla)
        if k >= V:  # every token of the vocabulary is in the top V
            in_vocab_everywhere = np.array([((tok[b] >= 0) & (tok[b] < V)).all() for b in range(B)])
            assert (r.accept_len[in_vocab_everywhere] == K).all()
            assert r.accept_len[0] == 2 and r.accept_len[1] == 1  # stops exactly at the ids outside the vocabulary
        assert (r.accept_len >= vanilla).all()
        if prev is not None:
            assert (r.accept_len >= prev).all()  # a larger K accepts more (Section 4.1)
        prev = r.accept_len.copy()
    r = orc.verify_topk(ht, W, tok, V, dtype)
    assert r.accept_len[0] == 2 and r.accept_len[1] == 1 and r.rank[0, 2] == V


# ------------------------------------------------------ sampling by the Gumbel-max trick (Appendix A)


def test_philox_known_answers():
    """Known-answer vectors of Philox4x32-10 as published with the Random123 library."""
    kat = [((0, 0, 0, 0), (0, 0), (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)),
           ((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0),
            (0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1))]
    for ctr, key, want in kat:
        assert tuple(int(x) for x in orc.philox4x32_10(ctr, key)) == want


def test_noise_is_a_uniform_in_the_open_interval_and_exact_in_fp32():
    us = np.array([orc.noise_uniform(7, 3, j, v) for j in range(8) for v in range(500)])
    assert (us > 0).all() and (us < 1).all()
    assert (us.astype(np.float32).astype(np.float64) == us).all()
    assert 0.45 < us.mean() < 0.55 and len(np.unique(us)) > 3990
    # rows 4q .. 4q+3 take the four words of one Philox call, and every argument matters
    base = orc.noise_uniform(7, 3, 5, 11)
    assert base == orc.noise_uniform(7, 3, 5, 11)
    assert len({base, orc.noise_uniform(8, 3, 5, 11), orc.noise_uniform(7, 4, 5, 11), orc.noise_uniform(7, 3, 6, 11),
                orc.noise_uniform(7, 3, 5, 12), orc.noise_uniform(7 + (1 << 32), 3, 5, 11), orc.noise_uniform(7, 3 + (1 << 32), 5, 11)}) == 7
    w = orc.philox4x32_10((11, 1, 3, 0), (7, 0))
    assert base == (float(int(w[1]) >> 9) + 0.5) / 8388608.0
    assert orc.gumbel(7, 3, 5, 11) == pytest.approx(-np.log(-np.log(base)), rel=1e-15)


def test_gumbel_max_draws_follow_the_softmax_and_zero_temperature_is_greedy():
    """Appendix A: adding independent Gumbel noise to the logits and taking the argmax draws an index with
    the softmax probabilities; at temperature T the distribution is softmax(logit / T)."""
    V, d, T = 6, 8, 0.7
    cfg = gen.Config("gumbel", B=1, K=3, d=d, d_draft=0, V=V, dtype=F32, sigma_W=0.6, seed=71)
    W = gen.make_W(cfg)
    ht, _ = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    tok = np.zeros((1, 3), np.int32)
    lg = orc.logits(ht[0], W, F32)                               # [4, V]
    greedy = orc.verify(ht, None, W, tok, w, 0.0, 0.5, F32)
    np.testing.assert_array_equal(greedy.target_tok[0], lg.argmax(1))
    again = orc.verify(ht, None, W, tok, w, 0.0, 0.5, F32, temperature=0.0, seed=99, step=5)
    np.testing.assert_array_equal(again.target_tok, greedy.target_tok)   # T = 0 ignores the random state
    n = 6000
    counts = np.zeros((4, V))
    for step in range(n):
        r = orc.verify(ht, None, W, tok, w, 0.0, 0.5, F32, temperature=T, seed=2024, step=step)
        for j in range(4):
            counts[j, r.target_tok[0, j]] += 1
    p = np.exp(lg / T)
    p /= p.sum(1, keepdims=True)
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum(1)              # 5 degrees of freedom per row
    assert (chi2 < 25.0).all(), chi2                             # P(chi2_5 > 25) = 1.4e-4
    same = orc.verify(ht, None, W, tok, w, 0.0, 0.5, F32, temperature=T, seed=2024, step=17)
    np.testing.assert_array_equal(same.target_tok, orc.verify(ht, None, W, tok, w, 0.0, 0.5, F32, temperature=T, seed=2024, step=17).target_tok)
    # the reported winner is the noisy score
    j, y = 2, int(same.target_tok[0, 2])
    assert same.top1[0, j] == pytest.approx(lg[j, y] + T * orc.gumbel(2024, 17, j, y), abs=1e-12)


# ------------------------------------------------------ tree drafts (Section 3.3 "Generality", EAGLE-2 appendix)


def _random_tree(rng, N, shape="random"):
    if shape == "chain":
        return np.arange(-1, N - 1, dtype=np.int32)
    if shape == "star":
        return np.full(N, -1, np.int32)
    return np.array([rng.integers(-1, n) for n in range(N)], dtype=np.int32)


def _paths(parent):
    """Root-to-node path (list of node indices, root excluded) of every node with a valid ancestry."""
    out = {}
    for n, q in enumerate(parent):
        if q == -1:
            out[n] = [n]
        elif 0 <= q < n and q in out:
            out[n] = out[q] + [n]
    return out


def test_tree_rule_is_the_window_rule_on_every_root_to_node_path():
    """Brute force: a node is accepted iff the window rule (the pinned accept walk) accepts the whole window
    formed by its root path; the result is the deepest such node, the lowest index among equals."""
    rng = np.random.default_rng(5)
    for trial in range(400):
        N = int(rng.integers(1, 9))
        parent = _random_tree(rng, N, ("random", "random", "chain", "star")[trial % 4])
        if trial % 7 == 3 and N > 2:
            parent[int(rng.integers(1, N))] = N + 3          # an invalid parent: that node and its subtree never count
        y = rng.integers(0, 3, N + 1).astype(np.int32)
        tok = rng.integers(0, 3, N).astype(np.int32)
        p = rng.random(N)
        tau = float(rng.choice([0.0, 0.3, 0.6, 1.0]))
        best, best_len = -1, 0
        for n, path in _paths(parent).items():
            rows = [0] + [m + 1 for m in path]               # the rows along the path, root first
            win_y = y[rows][None, :]                         # the window's target tokens
            win_tok = tok[path][None, :]
            win_p = p[path][None, :]
            acc, _ = orc.rewalk(win_y, win_tok, win_p, tau)
            if acc[0] == len(path) and len(path) > best_len:
                best, best_len = n, len(path)
        got = orc.tree_accept(tok, parent, y, p, tau)
        assert got == (best_len, best, int(y[best + 1])), (trial, parent, tok, y, p, tau, got, best)


def test_tree_rule_special_cases():
    y = np.array([5, 6, 7, 8, 9], np.int32)
    p = np.array([0.9, 0.2, 0.9, 0.2])
    chain = np.array([-1, 0, 1, 2], np.int32)
    # a chain is a window: stop at the first mismatch that is not forgiven
    assert orc.tree_accept([5, 6, 0, 8], chain, y, p, 0.5) == (2, 1, 7)
    assert orc.tree_accept([5, 0, 0, 8], chain, y, p, 0.5) == (2, 1, 7)     # node 1 forgiven (0.2 < 0.5), node 2 not
    assert orc.tree_accept([5, 0, 0, 8], chain, y, p, 0.0) == (1, 0, 6)     # nothing forgiven
    assert orc.tree_accept([0, 0, 0, 0], chain, y, p, 1.0) == (4, 3, 9)     # everything forgiven
    assert orc.tree_accept([0, 6, 7, 8], chain, y, p, 0.5) == (0, -1, 5)    # the first node fails: the root stands
    # a star: depth 1 at most, the first passing child wins
    star = np.full(4, -1, np.int32)
    assert orc.tree_accept([1, 2, 5, 5], star, y, p, 0.0) == (1, 2, 8)
    assert orc.tree_accept([1, 2, 3, 4], star, y, p, 0.5) == (1, 1, 7)
    # two branches: the deeper accepted one wins even if it comes later; equal depth: the lower index
    par = np.array([-1, -1, 1, 2], np.int32)
    assert orc.tree_accept([5, 5, 7, 8], par, y, p, 0.0) == (3, 3, 9)
    assert orc.tree_accept([5, 5, 0, 7], par, y, np.array([0.9, 0.9, 0.9, 0.9]), 0.5) == (1, 0, 6)
    # a match is tested against the PARENT's row: node 2 (child of node 1) must equal y[2]
    assert orc.tree_accept([5, 5, 7, 0], par, y, p, 0.0) == (2, 2, 8)
    assert orc.tree_accept([5, 5, 8, 0], par, y, np.array([0.9] * 4), 0.5) == (1, 0, 6)
    # accept_len never decreases with tau
    rng = np.random.default_rng(2)
    for _ in range(50):
        N = 7
        parent = _random_tree(rng, N)
        yy, tt, pp = rng.integers(0, 3, N + 1).astype(np.int32), rng.integers(0, 3, N).astype(np.int32), rng.random(N)
        lens = [orc.tree_accept(tt, parent, yy, pp, t)[0] for t in (0.0, 0.2, 0.5, 0.8, 1.0)]
        assert lens == sorted(lens)
        depth = {n: len(path) for n, path in _paths(parent).items()}
        assert lens[-1] == max(depth.values())


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_tree_step_reduces_to_the_window_step_on_a_chain_and_composes_from_its_parts(dtype):
    cfg = gen.Config("tree", B=3, K=6, d=40, d_draft=24, V=50, dtype=dtype, sigma_w=0.4, match_lo=0.4, match_hi=0.8, seed=81)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, dtype)] for b in range(cfg.B)])
    tok = gen.plant_draft_tokens(cfg, y)
    chain = np.tile(np.arange(-1, cfg.K - 1, dtype=np.int32), (cfg.B, 1))
    for tau in (0.0, 0.4, 0.7, 1.0):
        a = orc.verify(ht, hd, W, tok, w, cfg.judge_b, tau, dtype)
        t = orc.verify_tree(ht, hd, W, tok, chain, w, cfg.judge_b, tau, dtype)
        np.testing.assert_array_equal(t.accept_len, a.accept_len)
        np.testing.assert_array_equal(t.next_tok, a.next_tok)
        np.testing.assert_array_equal(t.target_tok, a.target_tok)
        np.testing.assert_array_equal(t.best_node, a.accept_len - 1)
        np.testing.assert_array_equal(t.judge_p, a.judge_p)
    # a real tree: tokens planted against the parents' rows; the step equals argmax + judge_p + the rule
    rng = np.random.default_rng(9)
    parent = np.stack([_random_tree(rng, cfg.K) for _ in range(cfg.B)])
    tok = np.stack([np.where(rng.random(cfg.K) < 0.7, y[b][parent[b] + 1], rng.integers(0, cfg.V, cfg.K)) for b in range(cfg.B)]).astype(np.int32)
    t = orc.verify_tree(ht, hd, W, tok, parent, w, cfg.judge_b, 0.5, dtype)
    np.testing.assert_array_equal(t.target_tok, y)
    for b in range(cfg.B):
        mism = tok[b] != y[b][parent[b] + 1]
        assert mism.any() and (~mism).any()
        assert (np.isnan(t.judge_p[b]) == ~mism).all()
        for n in np.nonzero(mism)[0]:
            assert t.judge_p[b, n] == orc.judge_p(hd[b, n + 1], ht[b, n + 1], dtype, w, cfg.judge_b)
        assert (t.accept_len[b], t.best_node[b], t.next_tok[b]) == orc.tree_accept(tok[b], parent[b], y[b], np.nan_to_num(t.judge_p[b]), 0.5)
    # sampled target tokens: the same rows and noise as the window step
    s = orc.verify_tree(ht, hd, W, tok, chain, w, cfg.judge_b, 0.5, dtype, temperature=0.8, seed=3, step=2)
    np.testing.assert_array_equal(s.target_tok, orc.verify(ht, hd, W, tok, w, cfg.judge_b, 0.5, dtype, temperature=0.8, seed=3, step=2).target_tok)


def test_a_slice_of_a_batch_draws_the_noise_of_its_own_rows():
    cfg = gen.Config("slice", B=4, K=3, d=16, d_draft=8, V=40, dtype=F32, sigma_W=0.5, sigma_w=0.3, seed=83)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    tok = gen.random_draft_tokens(cfg)
    full = orc.verify(ht, hd, W, tok, w, cfg.judge_b, 0.5, F32, temperature=1.1, seed=6, step=7)
    for b in range(cfg.B):
        one = orc.verify(ht[b : b + 1], hd[b : b + 1], W, tok[b : b + 1], w, cfg.judge_b, 0.5, F32, temperature=1.1, seed=6, step=7, row0=b * 4)
        np.testing.assert_array_equal(one.target_tok[0], full.target_tok[b])
        np.testing.assert_array_equal(one.top1[0], full.top1[b])
        assert one.accept_len[0] == full.accept_len[b]
    moved = orc.verify(ht[1:2], hd[1:2], W, tok[1:2], w, cfg.judge_b, 0.5, F32, temperature=1.1, seed=6, step=7, row0=0)
    assert (moved.top1[0] != full.top1[1]).any()
