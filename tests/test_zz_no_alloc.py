"""aj_verify_static, the entry point for callers that cannot allocate device memory (a server
that gave every byte to its own pool, an audited or frozen allocator): it must give what the
handle-based aj_verify gives, on two calls in a row that share its fixed scratch array.

Collected last on purpose, so a run that stops at the first failure has run everything else."""
import numpy as np
import pytest

import aj_inputs as gen

pytestmark = pytest.mark.gpu


def _both(cfg, seed_shift=0, expect_path=None):
    import torch

    import paper_2504_20039_b200 as aj
    from aj_testlib import DeviceCase, GpuResult, check_parity
    from oracle import aj_oracle as orc

    cfg = gen.scaled(cfg, seed=cfg.seed + seed_shift)
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        # draft tokens planted against the oracle's greedy tokens: a realistic mix of matches
        y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(cfg.B)])
        tok = gen.plant_draft_tokens(cfg, y)
        want = case.run(tok, cfg.tau)
        if expect_path:
            assert want.path == expect_path  # the kernel aj_verify chose; the static entry point makes the same choice

        i32 = dict(dtype=torch.int32, device="cuda")
        f32 = dict(dtype=torch.float32, device="cuda")
        tok_d = torch.from_numpy(tok).cuda()
        acc, nxt = torch.full((cfg.B,), -3, **i32), torch.full((cfg.B,), -3, **i32)
        tt = torch.full((cfg.B, cfg.K + 1), -3, **i32)
        top1, jp = torch.full((cfg.B, cfg.K + 1), 7.0, **f32), torch.full((cfg.B, cfg.K), 7.0, **f32)
        status = torch.full((1,), 99, **i32)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]  # what the driver has left: it counts every allocation of the process
        aj.verify_static(case.ht, case.hd, case.W, tok_d, case.w, cfg.judge_b, cfg.tau, cfg.B, cfg.K, cfg.d, cfg.d_draft,
                         cfg.V, cfg.dtype, aj.AJ_W_VD, acc, nxt, tt, top1, jp, status,
                         stream=torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # one more call, now that the first call on this device has done its set-up: no byte of device memory may go
        free_mid = torch.cuda.mem_get_info()[0]
        aj.verify_static(case.ht, case.hd, case.W, tok_d, case.w, cfg.judge_b, cfg.tau, cfg.B, cfg.K, cfg.d, cfg.d_draft,
                         cfg.V, cfg.dtype, aj.AJ_W_VD, acc, nxt, tt, top1, jp, status,
                         stream=torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_mid and free_mid <= free_before
        assert int(status.item()) == 0
        # against the oracle, under the tolerances of every other parity test
        got = GpuResult(acc.cpu().numpy(), nxt.cpu().numpy(), tt.cpu().numpy(), top1.cpu().numpy(), jp.cpu().numpy(), want.path, 2)
        check_parity(orc.verify(ht, hd, W, tok, w, cfg.judge_b, cfg.tau, cfg.dtype), got, tok, cfg.tau)
        np.testing.assert_array_equal(tt.cpu().numpy(), want.target_tok)
        np.testing.assert_array_equal(acc.cpu().numpy(), want.accept_len)
        np.testing.assert_array_equal(nxt.cpu().numpy(), want.next_tok)
        np.testing.assert_allclose(top1.cpu().numpy(), want.top1, rtol=0, atol=2e-2)
        np.testing.assert_allclose(jp.cpu().numpy(), want.judge_p, rtol=0, atol=1e-4, equal_nan=True)
    finally:
        case.close()


def test_static_scratch_entry_point_matches_handle_entry_point_twice():
    # first a larger batch, then a smaller one with other data: the second call finds the first
    # call's keys in the shared array and must not be disturbed by them
    big = gen.Config("static_a", B=5, K=40, d=512, d_draft=256, V=5000, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.9, seed=30)
    small = gen.Config("static_b", B=2, K=9, d=256, d_draft=128, V=3001, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.9, seed=31)
    _both(big, expect_path="umma_pair_256x256")   # 205 rows: the two-SM kernel, as aj_verify chooses
    _both(small, expect_path="umma_vm_128x32")
    _both(gen.scaled(small, dtype=gen.F32, d=200, d_draft=72), expect_path="simt")  # the CUDA-core kernel shares the same scratch
    wide = gen.Config("static_c", B=9, K=40, d=256, d_draft=128, V=3000, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.9, seed=32)
    _both(wide, expect_path="umma_pair_256x256")  # 369 rows: wide tiles on two accumulators


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    import torch

    import paper_2504_20039_b200 as aj

    i32 = dict(dtype=torch.int32, device="cuda")
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    t = torch.zeros(8, **i32)
    w = torch.zeros(64, dtype=torch.float32, device="cuda")
    too_many = aj.AJ_STATIC_MAX_ROWS // 2 + 1  # B * (K + 1) with K = 1
    st = aj.verify_static(x, None, x, t, w, 0.0, 0.5, too_many, 1, 64, 0, 1, aj.AJ_BF16, aj.AJ_W_VD, t, t, check=False)
    assert st == aj.AJ_ERR_WORKSPACE and "workspace" in aj.status_string(st)
    st = aj.verify_static(None, None, x, t, w, 0.0, 0.5, 1, 1, 64, 0, 1, aj.AJ_BF16, aj.AJ_W_VD, t, t, check=False)
    assert st == aj.AJ_ERR_INVALID_ARG
