"""The top-K rule (paper Section 4.1: accept a mismatching draft token iff it is among the target's top_k
tokens) on the CUDA library against the CPU oracle: ranks within the band of near-equal logits, accept
lengths exact wherever that band cannot move the decision."""
import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import DeviceCase, TOL_LOGIT, GAP_EXEMPT

pytestmark = pytest.mark.gpu

BAND = 1e-2  # logits closer than this to the draft token's may be ordered differently by fp32 arithmetic


def _orc():
    from oracle import aj_oracle as orc

    return orc


SHAPES = [
    # name, B, K, d, V, dtype, layout, flags, path
    ("one_sm", 3, 9, 256, 3000, gen.BF16, 0, 0, "umma_vm_128x32"),
    ("one_sm_wide", 6, 20, 192, 1000, gen.BF16, 0, 0, "umma_vm_128x128"),
    ("pair_single", 9, 63, 128, 2000, gen.BF16, 0, 0, "umma_pair_256x256"),
    ("pair_dual", 5, 60, 256, 5000, gen.BF16, 0, 0, "umma_pair_256x256"),
    ("dv_layout", 5, 60, 256, 5000, gen.BF16, 1, 0, "umma_pair_256x256"),
    ("cuda_cores_f32", 3, 9, 200, 1234, gen.F32, 0, 0, "simt"),
    ("cuda_cores_bf16", 2, 7, 128, 999, gen.BF16, 0, 1, "simt"),
]


@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_top_k_rule_matches_the_oracle(shape):
    orc = _orc()
    name, B, K, d, V, dtype, layout, flags, path = shape
    cfg = gen.Config(name, B=B, K=K, d=d, d_draft=0, V=V, dtype=dtype, sigma_W=0.2, match_lo=0.3, match_hi=0.8, seed=41)
    W = gen.make_W(cfg, layout)
    ht, _ = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, dtype, layout)] for b in range(B)])
    tok = gen.plant_draft_tokens(cfg, y)
    tok[0, min(2, K - 1)] = -4          # ids outside the vocabulary are never accepted
    tok[B - 1, 0] = V + 1
    case = DeviceCase(cfg, W, ht, None, w, layout=layout, flags=flags)
    try:
        for k in (1, 2, 8, 64, V):
            case.handle.set_top_k(k)
            o = orc.verify_topk(ht, W, tok, k, dtype, layout, band=BAND)
            g = case.run(tok, 0.5)
            assert g.path == path and g.launches == 3
            for b in range(B):
                ok_rows = o.gap[b] > GAP_EXEMPT
                assert (g.target_tok[b][ok_rows] == o.target_tok[b][ok_rows]).all()
                assert np.abs(g.top1[b] - o.top1[b]).max() <= TOL_LOGIT
                mism = o.rank[b] >= 0
                same = g.target_tok[b][:K] == o.target_tok[b][:K]
                assert (np.isnan(g.judge_p[b]) == ~mism)[same].all()
                in_vocab = (tok[b] >= 0) & (tok[b] < V)
                chk = mism & same
                # the device's rank agrees with the oracle's up to the entries too close to call, as long as it
                # is below top_k; the count of a rejected token stops somewhere from top_k up to its rank
                sel = chk & in_vocab
                got, want, near = g.judge_p[b][sel], o.rank[b][sel], o.near[b][sel]
                exact = want + near < k
                assert (np.abs(got - want) <= near)[exact].all()
                assert (got[~exact] >= np.minimum(k, want - near)[~exact]).all() and (got[~exact] <= (want + near)[~exact]).all()
                assert (g.judge_p[b][chk & ~in_vocab] == V).all()
                n = int(o.accept_len[b])
                upto = slice(0, min(n + 1, K))
                shaky = (mism[upto] & (np.abs(o.rank[b][upto] - k) <= o.near[b][upto]) & (o.near[b][upto] > 0)).any()
                if ok_rows[: n + 1].all() and not shaky:
                    assert g.accept_len[b] == n and g.next_tok[b] == o.next_tok[b], (name, k, b)
                assert g.next_tok[b] == g.target_tok[b, g.accept_len[b]]
            if k == 1:  # plain greedy verification
                first = np.array([int(np.argmax(np.append(tok[b] != g.target_tok[b, :K], True))) for b in range(B)])
                np.testing.assert_array_equal(g.accept_len, first)
        # back to the classifier: the handle behaves as before
        case.handle.set_top_k(0)
        g = case.run(tok, 0.0)
        assert g.launches == 2
        first = np.array([int(np.argmax(np.append(tok[b] != g.target_tok[b, :K], True))) for b in range(B)])
        np.testing.assert_array_equal(g.accept_len, first)
    finally:
        case.close()


def test_top_k_needs_no_classifier_operands_and_rejects_what_it_cannot_do():
    import torch

    import paper_2504_20039_b200 as aj

    h = aj.Handle(0, 2, 4, 128, 64, 1000)
    try:
        assert h.set_top_k(-1, check=False) == aj.AJ_ERR_INVALID_ARG
        h.set_top_k(4)
        x = torch.zeros((2, 5, 128), dtype=torch.bfloat16, device="cuda")
        Wl = torch.zeros((1000, 128), dtype=torch.bfloat16, device="cuda")
        t = torch.full((2, 4), 3, dtype=torch.int32, device="cuda")
        acc, nxt = torch.zeros(2, dtype=torch.int32, device="cuda"), torch.zeros(2, dtype=torch.int32, device="cuda")
        assert h.verify(x, None, Wl, t, None, 0.0, 0.0, 2, 4, acc, nxt) == aj.AJ_OK  # no judge_w, no h_draft
        torch.cuda.synchronize()
        # all logits are zero: the target's token is 0, draft token 3 has three entries ahead of it: rank 3 < 4
        assert (acc.cpu() == 4).all() and (nxt.cpu() == 0).all()
        h.set_top_k(3)
        assert h.verify(x, None, Wl, t, None, 0.0, 0.0, 2, 4, acc, nxt) == aj.AJ_OK
        torch.cuda.synchronize()
        assert (acc.cpu() == 0).all()
        assert h.last_status() == aj.AJ_OK
    finally:
        h.destroy()
    h = aj.Handle(0, 2, 4, 128, 64, 1000, flags=aj.AJ_FLAG_NO_EXTRA_ROW)
    try:
        assert h.set_top_k(2, check=False) == aj.AJ_ERR_UNSUPPORTED
    finally:
        h.destroy()
