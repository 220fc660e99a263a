"""Vocabulary-parallel form on ONE GPU: the ranks of a group are emulated as handles on the same device
whose exchange buffers all live there.  Every rank's projection (which publishes its keys into all
buffers) is enqueued before any rank's finish, so no kernel ever waits for a later one.  All ranks must
reproduce, bit for bit, what the unsharded handle gives, and that in turn matches the oracle."""
import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import DeviceCase, GpuResult, check_parity

pytestmark = pytest.mark.gpu


def _oracle():
    from oracle import aj_oracle as orc

    return orc


class ShardedGroup:
    def __init__(self, cfg, case: DeviceCase, world: int, ranges=None, flags: int = 0):
        import torch

        import paper_2504_20039_b200 as aj

        self.torch, self.aj, self.cfg, self.case, self.world = torch, aj, cfg, case, world
        nbytes = aj.shard_exchange_bytes(cfg.B, cfg.K, world)
        assert nbytes > 0
        # garbage, not zeros: creation must clear what matters
        self.bufs = [torch.full((nbytes // 8,), 0x7F7F7F7F7F7F7F7F, dtype=torch.int64, device="cuda") for _ in range(world)]
        self.ranges = ranges or [aj.shard_range(cfg.V, world, r) for r in range(world)]
        self.handles = [aj.Handle(0, cfg.B, cfg.K, cfg.d, cfg.d_draft, cfg.V, cfg.dtype, aj.AJ_W_VD, flags,
                                  shard=(r, world, self.ranges[r][0], self.ranges[r][1], self.bufs)) for r in range(world)]
        self.shards = [case.W[b : b + n] for b, n in self.ranges]  # contiguous row slices of W_lm

    def cycle(self, tok, tau, B=None, K=None, order=None):
        torch, cfg, case = self.torch, self.cfg, self.case
        B, K = B or cfg.B, K or cfg.K
        stream = torch.cuda.current_stream().cuda_stream
        tok_d = torch.from_numpy(np.ascontiguousarray(tok, dtype=np.int32)).cuda()
        ht = case.ht[:B, : K + 1].contiguous()
        hd = None if case.hd is None else case.hd[:B, : K + 1].contiguous()
        order = list(range(self.world)) if order is None else order
        for r in order:  # every projection first ...
            self.handles[r].shard_project(ht, self.shards[r], B, K, stream=stream)
        outs = []
        for r in range(self.world):  # ... then every finish: all flags are already set
            i32, f32 = dict(dtype=torch.int32, device="cuda"), dict(dtype=torch.float32, device="cuda")
            o = [torch.full((B,), -7, **i32), torch.full((B,), -7, **i32), torch.full((B, K + 1), -7, **i32),
                 torch.full((B, K + 1), 9.0, **f32), torch.full((B, K), 9.0, **f32)]
            self.handles[r].shard_finish(ht, hd, tok_d, case.w, cfg.judge_b, tau, B, K, *o, stream=stream)
            outs.append(o)
        torch.cuda.synchronize()
        res = []
        for r, o in enumerate(outs):
            assert self.handles[r].last_status() == self.aj.AJ_OK
            res.append(GpuResult(*[x.cpu().numpy() for x in o], self.handles[r].last_gemm_path(), self.handles[r].last_launch_count()))
        return res

    def close(self):
        for h in self.handles:
            h.destroy()


def _same(a: GpuResult, b: GpuResult):
    np.testing.assert_array_equal(a.target_tok, b.target_tok)
    np.testing.assert_array_equal(a.accept_len, b.accept_len)
    np.testing.assert_array_equal(a.next_tok, b.next_tok)
    np.testing.assert_array_equal(a.top1, b.top1)  # the same logits, bit for bit: no split over k
    np.testing.assert_array_equal(a.judge_p, b.judge_p)


CASES = [
    # name, B, K, d, d_draft, V, world
    ("two_ranks_small_m", 2, 7, 256, 128, 5000, 2),         # one-SM kernel, 20 blocks of 256 -> 10 + 10
    ("three_ranks_uneven", 3, 20, 128, 64, 3000, 3),        # 12 blocks -> 4 + 4 + 4, last shard ragged (3000 = 11*256 + 184)
    ("eight_ranks_pair_kernel", 5, 60, 256, 128, 9001, 8),  # M = 305: two-SM kernel; 36 blocks -> 5,5,5,5,4,4,4,4
    ("one_rank", 2, 5, 128, 0, 700, 1),                     # a group of one: publish to and gather from the own buffer
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_every_rank_reproduces_the_unsharded_result(case):
    orc = _oracle()
    name, B, K, d, dd, V, world = case
    cfg = gen.Config(name, B=B, K=K, d=d, d_draft=dd, V=V, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.95, seed=21)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(B)])
    tok = gen.plant_draft_tokens(cfg, y)
    one = DeviceCase(cfg, W, ht, hd, w)
    grp = ShardedGroup(cfg, one, world)
    try:
        assert sum(n for _, n in grp.ranges) == V and grp.ranges[0][0] == 0
        for cycle, tau in enumerate((0.5, 0.0, 1.0, 0.3)):  # several cycles: epochs and both slot parities
            want = one.run(tok, tau)
            o = orc.verify(ht, hd, W, tok, w, cfg.judge_b, tau, cfg.dtype)
            check_parity(o, want, tok, tau)
            got = grp.cycle(tok, tau, order=list(range(world))[:: 1 if cycle % 2 == 0 else -1])
            for r in range(world):
                _same(got[r], want)
                assert got[r].launches == 2
    finally:
        grp.close()
        one.close()


def test_fp32_storage_shards_on_the_cuda_core_kernel():
    orc = _oracle()
    cfg = gen.Config("f32_shards", B=2, K=6, d=72, d_draft=40, V=1100, dtype=gen.F32, sigma_w=0.05, seed=23)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(cfg.B)])
    tok = gen.plant_draft_tokens(cfg, y)
    one = DeviceCase(cfg, W, ht, hd, w)
    grp = ShardedGroup(cfg, one, 3)
    try:
        want = one.run(tok, 0.5)
        check_parity(orc.verify(ht, hd, W, tok, w, cfg.judge_b, 0.5, cfg.dtype), want, tok, 0.5)
        for g in grp.cycle(tok, 0.5):
            assert g.path == "simt"
            np.testing.assert_array_equal(g.target_tok, want.target_tok)
            np.testing.assert_array_equal(g.accept_len, want.accept_len)
            np.testing.assert_array_equal(g.next_tok, want.next_tok)
            np.testing.assert_allclose(g.top1, want.top1, rtol=0, atol=1e-5)  # other warp slices: other summation order
    finally:
        grp.close()
        one.close()


def test_smaller_batch_after_a_larger_one_and_winner_in_every_shard():
    # Plant the winner of chosen rows in a chosen shard; then reuse the group for a smaller batch,
    # so stale keys of the larger cycle sit in the slots beyond the rows in use.
    orc = _oracle()
    cfg = gen.Config("planted", B=4, K=9, d=128, d_draft=64, V=2048, sigma_W=0.05, sigma_w=0.05, seed=22)
    W = gen.make_W(cfg).copy()
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    world = 4
    # row j of sequence 0 wins in shard j % 4: W[v] = 4 * that row (exact in bf16)
    hf = gen.bf16_bits_to_f32(ht)
    for j in range(cfg.K + 1):
        v = (j % world) * 512 + 17 + j
        W[v] = gen.f32_to_bf16_bits(hf[0, j] * 4.0)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(cfg.B)])
    assert [int(v) // 512 for v in y[0]] == [j % world for j in range(cfg.K + 1)]
    tok = gen.plant_draft_tokens(cfg, y)
    one = DeviceCase(cfg, W, ht, hd, w)
    grp = ShardedGroup(cfg, one, world)
    try:
        want = one.run(tok, 0.5)
        for g in grp.cycle(tok, 0.5):
            _same(g, want)
        np.testing.assert_array_equal(want.target_tok, y)
        # the unsharded reference for a smaller call reads rows [:2, :5] of the hidden states
        cfg_s = gen.scaled(cfg, B=2, K=4)
        ref = DeviceCase(cfg_s, one.W, ht[:2, :5].copy(), hd[:2, :5].copy(), w)
        try:
            want_s = ref.run(tok[:2, :4], 0.5)
        finally:
            ref.close()
        for g in grp.cycle(tok[:2, :4], 0.5, B=2, K=4):
            _same(g, want_s)
    finally:
        grp.close()
        one.close()


def test_sharded_argument_checks():
    import torch

    import paper_2504_20039_b200 as aj

    buf = torch.zeros(aj.shard_exchange_bytes(2, 4, 2) // 8, dtype=torch.int64, device="cuda")
    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 2, 4, 128, 64, 1000, shard=(2, 2, 0, 500, [buf, buf]))  # rank out of range
    assert e.value.status == aj.AJ_ERR_INVALID_ARG
    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 2, 4, 128, 64, 1000, shard=(0, 2, 600, 500, [buf, buf]))  # range beyond the vocabulary
    assert e.value.status == aj.AJ_ERR_INVALID_ARG
    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 2, 4, 128, 64, 1000, shard=(0, 2, 0, 500, [buf, None]))
    assert e.value.status == aj.AJ_ERR_INVALID_ARG
    h = aj.Handle(0, 2, 4, 128, 64, 1000, shard=(0, 1, 0, 1000, [buf]))
    try:
        x = torch.zeros((2, 5, 128), dtype=torch.bfloat16, device="cuda")
        xd = torch.zeros((2, 5, 64), dtype=torch.bfloat16, device="cuda")
        t = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
        wj = torch.zeros(192, dtype=torch.float32, device="cuda")
        acc, nxt = torch.zeros(2, dtype=torch.int32, device="cuda"), torch.zeros(2, dtype=torch.int32, device="cuda")
        # a finish without its projection; two projections in a row
        assert h.shard_finish(x, xd, t, wj, 0.0, 0.5, 2, 4, acc, nxt, check=False) == aj.AJ_ERR_INVALID_ARG
        Wl = torch.zeros((1000, 128), dtype=torch.bfloat16, device="cuda")
        assert h.shard_project(x, Wl, 2, 4) == aj.AJ_OK
        assert h.shard_project(x, Wl, 2, 4, check=False) == aj.AJ_ERR_INVALID_ARG
        assert h.verify(x, xd, Wl, t, wj, 0.0, 0.5, 2, 4, acc, nxt, check=False) == aj.AJ_ERR_INVALID_ARG
        assert h.shard_finish(x, xd, t, wj, 0.0, 0.5, 2, 4, acc, nxt) == aj.AJ_OK
        assert h.verify(x, xd, Wl, t, wj, 0.0, 0.5, 2, 4, acc, nxt) == aj.AJ_OK  # a whole cycle on a group of one
        torch.cuda.synchronize()
        assert h.last_status() == aj.AJ_OK
        assert (acc.cpu() == 4).all() and (nxt.cpu() == 0).all()  # all logits zero: token 0 everywhere, everything matches
    finally:
        h.destroy()
    plain = aj.Handle(0, 2, 4, 128, 64, 1000)
    try:
        assert plain.shard_project(buf, buf, 1, 1, check=False) == aj.AJ_ERR_INVALID_ARG  # not a sharded handle
    finally:
        plain.destroy()


def test_a_rank_that_never_publishes_is_reported_as_a_timeout_and_the_gpu_stays_usable():
    """Failure detection without a fault: in a group of two, only rank 0 runs its cycle.  Nothing ever
    sets rank 1's flag in rank 0's exchange buffer, so rank 0's judge kernel gives up after its bounded
    wait (2 s), records AJ_ERR_TIMEOUT in the status word and returns normally."""
    import time

    import torch

    import paper_2504_20039_b200 as aj

    cfg = gen.Config("absent_peer", B=2, K=4, d=128, d_draft=64, V=1024, sigma_W=0.2, sigma_w=0.05, seed=24)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    tok = gen.random_draft_tokens(cfg)
    one = DeviceCase(cfg, W, ht, hd, w)
    grp = ShardedGroup(cfg, one, 2)
    try:
        want = one.run(tok, 0.5)
        h0 = grp.handles[0]
        i32 = dict(dtype=torch.int32, device="cuda")
        acc, nxt = torch.full((cfg.B,), -7, **i32), torch.full((cfg.B,), -7, **i32)
        t0 = time.time()
        h0.verify(one.ht, one.hd, grp.shards[0], torch.from_numpy(tok).cuda(), one.w, cfg.judge_b, 0.5, cfg.B, cfg.K, acc, nxt)
        torch.cuda.synchronize()  # returns: the wait is bounded
        waited = time.time() - t0
        assert 1.5 < waited < 20.0
        assert h0.last_status() == aj.AJ_ERR_TIMEOUT
        assert h0.last_status() == aj.AJ_OK  # reading the status clears it
        assert ((acc.cpu() >= 0) & (acc.cpu() <= cfg.K)).all()  # outputs are invalid but in range: nothing ran wild
    finally:
        grp.close()
    try:
        again = one.run(tok, 0.5)  # the context is intact: an ordinary cycle gives what it gave before
        np.testing.assert_array_equal(again.target_tok, want.target_tok)
        np.testing.assert_array_equal(again.accept_len, want.accept_len)
    finally:
        one.close()
