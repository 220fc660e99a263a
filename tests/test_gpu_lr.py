"""Fitting the classifier on the GPU (paper Section 3.2 / 4.1: L2-regularised logistic regression) against the
CPU oracle's minimiser: the fitted weights, the probabilities they give, and the judge kernel using them."""
import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import to_device

pytestmark = pytest.mark.gpu


def _fit(X, y, dtype, C, max_iter=500, tol=1e-7):
    import torch

    import paper_2504_20039_b200 as aj

    n, F = X.shape
    Xd = to_device(X, dtype)
    yd = torch.from_numpy(y).cuda()
    w = torch.full((F,), 7.0, dtype=torch.float32, device="cuda")
    st, b, iters, evals, gnorm = aj.lr_fit(0, Xd, yd, n, F, dtype, C, w, max_iter=max_iter, tol=tol)
    torch.cuda.synchronize()
    return w.cpu().numpy().astype(np.float64), float(b), iters, evals, gnorm


CASES = [
    # name, n, F, dtype, C
    ("small_f32", 500, 16, gen.F32, 1.0),
    ("ragged_rows_bf16", 1003, 64, gen.BF16, 1e-2),       # n is not a multiple of the row block
    ("many_rows_bf16", 20011, 256, gen.BF16, 1e-3),
    ("judge_width_bf16", 3000, 6144, gen.BF16, 1e-4),     # d_draft + d of the 1B / 8B pair, the paper's C
    ("few_rows", 5, 8, gen.BF16, 1.0),                    # fewer rows than there are warp groups
    ("f32_two_warps_per_row", 600, 1024, gen.F32, 1e-2),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_fit_reaches_the_oracles_minimiser(case):
    from oracle import aj_lr_oracle as lro

    name, n, F, dtype, C = case
    X, y = gen.make_labelled_features(n, F, dtype, seed=31)
    if name == "few_rows":
        y[:] = [1, 0, 0, 1, 0]
    Xf = gen.to_f64(X, dtype)
    w_o, b_o = lro.fit(Xf, y, C)
    w_g, b_g, iters, evals, gnorm = _fit(X, y, dtype, C)
    assert 1 <= iters <= 500 and evals >= iters
    # the gradient of the objective at the device's result, evaluated by the oracle in fp64
    _, gw, gb = lro.objective(Xf, y, C, w_g, b_g)
    scale = max(1.0, C * n)
    assert max(np.abs(gw).max(), abs(gb)) <= 2e-5 * scale, (iters, evals, gnorm, np.abs(gw).max(), gb)
    # the minimiser is unique: weights, intercept and the probabilities the judge would compute
    assert np.abs(w_g - w_o).max() <= 1e-3 * np.abs(w_o).max() + 1e-6, (np.abs(w_g - w_o).max(), np.abs(w_o).max())
    assert abs(b_g - b_o) <= 2e-3
    p_o, p_g = lro.predict_proba(Xf, w_o, b_o), lro.predict_proba(Xf, w_g, b_g)
    assert np.abs(p_o - p_g).max() <= 1e-3
    # and the objective value is the oracle's to 1e-6 relative
    f_o, f_g = lro.objective(Xf, y, C, w_o, b_o)[0], lro.objective(Xf, y, C, w_g, b_g)[0]
    assert f_o - 1e-12 <= f_g <= f_o * (1 + 1e-6) + 1e-9


def test_fit_is_reproducible_and_feeds_the_judge():
    """Two fits give the same bits (fixed-order reductions); the fitted weights drive aj_verify like any judge_w."""
    import torch

    import paper_2504_20039_b200 as aj
    from oracle import aj_oracle as orc

    cfg = gen.Config("lr_judge", B=2, K=6, d=64, d_draft=64, V=512, sigma_W=0.3, seed=33)
    F = cfg.d + cfg.d_draft
    X, y = gen.make_labelled_features(4000, F, gen.BF16, seed=35)
    a = _fit(X, y, gen.BF16, 1e-2)
    b = _fit(X, y, gen.BF16, 1e-2)
    np.testing.assert_array_equal(a[0], b[0])
    assert a[1] == b[1] and a[2:4] == b[2:4]
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    tok = gen.random_draft_tokens(cfg)
    w32 = a[0].astype(np.float32)
    o = orc.verify(ht, hd, W, tok, w32, a[1], 0.5, gen.BF16)
    from aj_testlib import DeviceCase, check_parity

    case = DeviceCase(cfg, W, ht, hd, w32)
    try:
        g = case.run(tok, 0.5, judge_b=a[1])
        check_parity(o, g, tok, 0.5)
        assert (~np.isnan(g.judge_p)).sum() > 5
    finally:
        case.close()


def test_fit_refuses_bad_arguments():
    import torch

    import paper_2504_20039_b200 as aj

    X = torch.zeros((8, 16), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(8, dtype=torch.uint8, device="cuda")
    w = torch.zeros(16, dtype=torch.float32, device="cuda")
    assert aj.lr_fit(0, X, y, 8, 16, aj.AJ_BF16, 0.0, w, check=False)[0] == aj.AJ_ERR_INVALID_ARG      # C must be positive
    assert aj.lr_fit(0, X, y, 0, 16, aj.AJ_BF16, 1.0, w, check=False)[0] == aj.AJ_ERR_INVALID_ARG
    assert aj.lr_fit(0, None, y, 8, 16, aj.AJ_BF16, 1.0, w, check=False)[0] == aj.AJ_ERR_INVALID_ARG
    assert aj.lr_fit(0, X, y, 8, 12, aj.AJ_BF16, 1.0, w, check=False)[0] == aj.AJ_ERR_UNSUPPORTED      # rows of 24 bytes
    wide = torch.zeros((4, 32768), dtype=torch.bfloat16, device="cuda")
    assert aj.lr_fit(0, wide, y, 4, 32768, aj.AJ_BF16, 1.0, torch.zeros(32768, device="cuda"), check=False)[0] == aj.AJ_ERR_UNSUPPORTED
    assert aj.lr_fit(0, X, y, 8, 16, aj.AJ_BF16, 1.0, w, check=False)[0] == aj.AJ_OK


def test_widest_rows_reach_a_stationary_point():
    """Rows of 48 KB (all 16 warps of a CTA on one row): too wide for the oracle's Newton steps, so the result is
    certified instead: the objective is strongly convex (modulus 1 in w), hence |w - w*| <= |gradient| at w,
    and the oracle evaluates that gradient in fp64."""
    from oracle import aj_lr_oracle as lro

    n, F, C = 300, 24576, 1e-3
    X, y = gen.make_labelled_features(n, F, gen.BF16, seed=37)
    w, b, iters, evals, gnorm = _fit(X, y, gen.BF16, C)
    Xf = gen.to_f64(X, gen.BF16)
    _, gw, gb = lro.objective(Xf, y, C, w, b)
    assert np.linalg.norm(gw) <= 1e-4 and abs(gb) <= 1e-5, (np.linalg.norm(gw), gb, iters, evals, gnorm)
    p = lro.predict_proba(Xf, w, b)
    assert p[y == 1].mean() > p[y == 0].mean()
