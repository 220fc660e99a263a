"""The two-SM projection kernel shares its tiles out through a counter in the handle's workspace
(the pairs take tiles in order as they become free; the pair that leaves last puts the counter back).
What that must not change: the result of a launch does not depend on which pair computed which tile,
launches enqueued back to back find the counter clean whatever shapes they alternate between, and
two handles have counters of their own, so their launches may overlap on the device."""
import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import DeviceCase, check_parity

pytestmark = pytest.mark.gpu


def _oracle():
    from oracle import aj_oracle as orc

    return orc


def _case(seed, B=10, K=59, d=128, V=60000):
    orc = _oracle()
    cfg = gen.Config(f"counter_{seed}", B=B, K=K, d=d, d_draft=64, V=V, sigma_W=0.2, sigma_w=0.05, match_lo=0.4, match_hi=0.9, seed=seed)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(cfg.B)])
    tok = gen.plant_draft_tokens(cfg, y)
    return cfg, W, ht, hd, w, tok


class _Outputs:
    def __init__(self, torch, B, K):
        self.acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        self.nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        self.tt = torch.full((B, K + 1), -7, dtype=torch.int32, device="cuda")
        self.jp = torch.full((B, K), 12345.0, dtype=torch.float32, device="cuda")

    def host(self):
        return self.acc.cpu().numpy(), self.nxt.cpu().numpy(), self.tt.cpu().numpy(), self.jp.cpu().numpy()


def _enqueue(case, tok_d, B, tau, out, stream):
    cfg = case.cfg
    case.handle.verify(case.ht[:B].contiguous(), case.hd[:B].contiguous(), case.W, tok_d[:B].contiguous(), case.w, cfg.judge_b, tau,
                       B, cfg.K, out.acc, out.nxt, out.tt, None, out.jp, stream=stream)


def test_back_to_back_launches_of_changing_shape():
    """Forty launches enqueued without a host synchronisation between them, alternating between a batch of
    600 rows (wide tiles, two row tiles per vocabulary block), 300 rows (one wide tile), 180 rows (narrow
    tiles) and 60 rows (the one-SM kernel, which has no counter): every launch of a shape gives the bits
    of the first launch of that shape, which is checked against the oracle."""
    import torch

    orc = _oracle()
    cfg, W, ht, hd, w, tok = _case(41)
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        tok_d = torch.from_numpy(tok.astype(np.int32)).cuda()
        stream = torch.cuda.current_stream().cuda_stream
        shapes = [10, 5, 3, 1]
        outs = []
        for i in range(40):
            B = shapes[i % len(shapes)] if i % 7 else shapes[(i // 7) % len(shapes)]
            out = _Outputs(torch, B, cfg.K)
            _enqueue(case, tok_d, B, 0.5, out, stream)
            outs.append((B, out))
        torch.cuda.synchronize()
        assert case.handle.last_status() == case.aj.AJ_OK
        first = {}
        for B, out in outs:
            got = out.host()
            if B not in first:
                first[B] = got
                o = orc.verify(ht[:B], hd[:B], W, tok[:B], w, cfg.judge_b, 0.5, cfg.dtype)
                g = case.run(tok[:B], 0.5, seqs=slice(0, B))
                check_parity(o, g, tok[:B], 0.5)
                np.testing.assert_array_equal(got[2], g.target_tok)
                np.testing.assert_array_equal(got[0], g.accept_len)
            for a, b in zip(got, first[B]):
                np.testing.assert_array_equal(a, b)
        assert sorted(first) == [1, 3, 5, 10]
    finally:
        case.close()


def test_two_handles_whose_launches_overlap():
    """Two handles on two streams, twenty launches each with nothing ordering one stream after the other:
    each handle's pairs draw from that handle's own counter."""
    import torch

    orc = _oracle()
    cases, toks, hosts = [], [], []
    try:
        for seed, B in ((42, 10), (43, 6)):
            cfg, W, ht, hd, w, tok = _case(seed, B=B)
            cases.append(DeviceCase(cfg, W, ht, hd, w))
            toks.append(torch.from_numpy(tok.astype(np.int32)).cuda())
            hosts.append((ht, hd, W, w, tok))
        torch.cuda.synchronize()
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        # the outputs are filled on the default stream: all of them first, so that no fill runs beside a launch
        outs = [[_Outputs(torch, case.cfg.B, case.cfg.K) for _ in range(20)] for case in cases]
        torch.cuda.synchronize()
        for i in range(20):
            for j, case in enumerate(cases):
                _enqueue(case, toks[j], case.cfg.B, 0.5, outs[j][i], streams[j].cuda_stream)
        torch.cuda.synchronize()
        for j, case in enumerate(cases):
            assert case.handle.last_status() == case.aj.AJ_OK
            ht, hd, W, w, tok = hosts[j]
            o = orc.verify(ht, hd, W, tok, w, case.cfg.judge_b, 0.5, case.cfg.dtype)
            g = case.run(tok, 0.5)
            assert g.path == "umma_pair_256x256"
            check_parity(o, g, tok, 0.5)
            for out in outs[j]:
                acc, nxt, tt, jp = out.host()
                np.testing.assert_array_equal(tt, g.target_tok)
                np.testing.assert_array_equal(acc, g.accept_len)
                np.testing.assert_array_equal(nxt, g.next_tok)
                np.testing.assert_array_equal(jp, g.judge_p)
    finally:
        for case in cases:
            case.close()
