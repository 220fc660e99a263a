"""GPU parity: the CUDA library, called through the C-ABI binding, against the CPU oracle on
the same seeded inputs, element by element.  Tolerances are in aj_testlib."""
import json
import os

import numpy as np
import pytest

import aj_inputs as gen
from aj_testlib import DeviceCase, check_parity, check_self_consistency

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


def _oracle():
    from oracle import aj_oracle as orc

    return orc


def _host_case(cfg, layout=0):
    W = gen.make_W(cfg, layout)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    return W, ht, hd, w


def _oracle_y(cfg, W, ht, layout=0, seqs=None):
    orc = _oracle()
    seqs = range(cfg.B) if seqs is None else seqs
    return np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype, layout)] for b in seqs])


def _full_parity(cfg, taus, flags=0, layout=0, expect_path=None):
    orc = _oracle()
    W, ht, hd, w = _host_case(cfg, layout)
    y = _oracle_y(cfg, W, ht, layout)
    tok = gen.plant_draft_tokens(cfg, y)
    case = DeviceCase(cfg, W, ht, hd, w, layout=layout, flags=flags)
    try:
        reports = []
        for tau in taus:
            o = orc.verify(ht, hd, W, tok, w, cfg.judge_b, tau, cfg.dtype, layout)
            g = case.run(tok, tau)
            if expect_path:
                assert g.path == expect_path
            assert g.launches == 2
            reports.append(check_parity(o, g, tok, tau))
            check_self_consistency(g, tok, tau, cfg.V)
        return reports
    finally:
        case.close()


# ------------------------------------------------------------------ small and cut-down shapes


@pytest.mark.parametrize("name", ["c1_tiny_f32", "tiny_bf16_b3"])
def test_golden_workloads(name):
    """The tiny workloads against the stored oracle values (tests/golden, written from the oracle)."""
    import importlib.util

    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    cfg = mg.CASES[name]
    with open(os.path.join(HERE, "golden", f"{name}.json")) as f:
        want = json.load(f)
    W, ht, hd, w = _host_case(cfg)
    tok = np.array(want["draft_tok"], np.int32)
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        g = case.run(tok, cfg.tau)
    finally:
        case.close()
    assert g.path == ("simt" if cfg.dtype == gen.F32 else "umma_vm_128x32")
    np.testing.assert_array_equal(g.target_tok, np.array(want["target_tok"]))
    np.testing.assert_array_equal(g.accept_len, np.array(want["accept_len"]))
    np.testing.assert_array_equal(g.next_tok, np.array(want["next_tok"]))
    np.testing.assert_allclose(g.top1, np.array(want["top1"]), rtol=0, atol=2e-2)
    wp = np.array([[np.nan if x is None else x for x in row] for row in want["judge_p"]])
    np.testing.assert_allclose(g.judge_p, wp, rtol=0, atol=1e-4, equal_nan=True)


SHAPES = [
    # name, B, K, d, d_draft, V : rows span several 128-row tiles with a ragged tail, V has a ragged tail
    ("one_row_tile", 1, 16, 1024, 512, 3000),
    ("three_row_tiles", 5, 60, 512, 256, 5000),   # M = 305 = 2*128 + 49, V = 19*256 + 136
    ("exact_tiles", 4, 31, 256, 128, 2048),       # M = 128, V = 16*128
    ("many_vocab_tiles", 3, 7, 128, 64, 70001),   # more vocabulary tiles than SMs, odd tail
    ("v_below_one_tile", 2, 3, 64, 64, 100),
    ("window_above_64", 2, 100, 64, 0, 700),      # K > 64: several ballots; target-only features
    ("pair_ragged_rows", 9, 63, 320, 64, 3000),   # M = 576 = 2*256 + 64: a 64-row tail tile on the two-SM kernel; V = 11*256 + 184
    ("pair_odd_tail", 3, 86, 192, 0, 1111),       # M = 261: 17 units of 16 rows on two accumulators (144 + 128), 3 k-blocks
    ("pair_two_full_tiles", 8, 63, 128, 64, 2000),  # M = 512: two tiles of 256 rows, one accumulator each
    ("pair_dual_448", 7, 63, 128, 64, 2000),      # M = 448: the largest batch on two accumulators (224 + 224)
    ("pair_dual_mid", 7, 56, 256, 0, 1500),       # M = 399: 25 units -> 208 + 192 rows
    ("pair_three_tiles", 11, 47, 128, 64, 1300),  # M = 528: just past the two-accumulator range, 3 tiles of 176 rows
    ("pair_dual_deep", 16, 64, 8192, 0, 700),     # M = 1040, d = 8192: deep contraction, two accumulators per tile (3 tiles)
]


@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
@pytest.mark.parametrize("flags", [0, 8, 1], ids=["umma_default", "umma_one_sm", "simt"])
def test_cut_down_shapes_bf16(shape, flags):
    name, B, K, d, dd, V = shape
    cfg = gen.Config(name, B=B, K=K, d=d, d_draft=dd, V=V, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.95, seed=3)
    reps = _full_parity(cfg, (0.0, 0.3, 0.5, 1.0), flags=flags)
    assert all(r.seqs_exempt <= r.seqs // 2 + 1 for r in reps)


MANY_TILES = [
    # name, B, K, flags, kernel: a vocabulary of 60000 entries gives every CTA (or CTA pair) at least three
    # tiles, so the alternation of the accumulator buffers, the wrap of the ring's phases from tile to
    # tile and the write-back of the running maxima on a change of row tile are exercised for every
    # tile width, not only the narrowest
    ("vm64_many_tiles", 1, 39, 0, "umma_vm_128x64"),        # M = 40: 469 tiles of 128 entries on 148 CTAs
    ("vm128_many_tiles", 4, 24, 0, "umma_vm_128x128"),      # M = 100
    ("vm256_many_tiles", 5, 59, 8, "umma_vm_128x256"),      # M = 300 on the one-SM kernel: two row tiles (256 + 48 rows)
    ("pair_narrow_many_tiles", 5, 39, 0, "umma_pair_256x256"),  # M = 200: 235 narrow tiles on 74 pairs
    ("pair_wide_many_tiles", 5, 59, 0, "umma_pair_256x256"),    # M = 300: 235 wide tiles (160 + 144 rows)
    ("pair_wide_two_row_tiles", 10, 59, 0, "umma_pair_256x256"),  # M = 600: 470 wide tiles, two row tiles (160 + 144 rows each)
]


@pytest.mark.parametrize("shape", MANY_TILES, ids=[s[0] for s in MANY_TILES])
def test_every_kernel_walks_several_tiles_per_cta(shape):
    name, B, K, flags, path = shape
    cfg = gen.Config(name, B=B, K=K, d=128, d_draft=64, V=60000, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.95, seed=21)
    reps = _full_parity(cfg, (0.0, 0.5, 1.0), flags=flags, expect_path=path)
    assert all(r.seqs_exempt <= r.seqs // 2 + 1 for r in reps)


def test_largest_window_the_interface_accepts():
    """K = 1024, the largest window a handle may be created for: the scan kernel's shared-memory
    layout there needs four bytes more than the default limit."""
    cfg = gen.Config("k1024", B=2, K=1024, d=64, d_draft=64, V=300, sigma_W=0.2, sigma_w=0.05, match_lo=0.9, match_hi=0.99, seed=22)
    _full_parity(cfg, (0.0, 0.5, 1.0))


@pytest.mark.parametrize("layout", [0, 1])
def test_fp32_storage_and_both_layouts(layout):
    cfg = gen.Config("f32", B=3, K=9, d=200, d_draft=72, V=1234, dtype=gen.F32, sigma_w=0.05, match_lo=0.6, match_hi=0.9, seed=4)
    _full_parity(cfg, (0.0, 0.5, 1.0), layout=layout, expect_path="simt")


@pytest.mark.parametrize("shape", [("dv_one_sm", 1, 16, 256, 128, 3000, "umma_vm_128x32"),
                                   ("dv_one_sm_wide", 6, 20, 192, 64, 1000, "umma_vm_128x128"),
                                   ("dv_pair_dual", 5, 60, 256, 128, 5000, "umma_pair_256x256"),
                                   ("dv_pair_single", 9, 63, 128, 64, 2000, "umma_pair_256x256")], ids=lambda s: s[0])
def test_bf16_dv_layout_on_the_tensor_cores(shape):
    """W_lm stored [d, V] (vocabulary entries contiguous) with V a multiple of 8: the tensor-core kernels
    read it as an MN-major operand; results must equal those of the [V, d] layout bit for bit."""
    name, B, K, d, dd, V, path = shape
    cfg = gen.Config(name, B=B, K=K, d=d, d_draft=dd, V=V, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.95, seed=15)
    reps = _full_parity(cfg, (0.0, 0.5, 1.0), layout=1, expect_path=path)
    assert all(r.seqs_exempt <= r.seqs // 2 + 1 for r in reps)
    W, ht, hd, w = _host_case(cfg, 0)
    tok = gen.random_draft_tokens(cfg)
    a = DeviceCase(cfg, W, ht, hd, w, layout=0)
    b = DeviceCase(cfg, np.ascontiguousarray(W.T), ht, hd, w, layout=1)
    try:
        ra, rb = a.run(tok, 0.5), b.run(tok, 0.5)
        np.testing.assert_array_equal(ra.target_tok, rb.target_tok)
        np.testing.assert_array_equal(ra.top1, rb.top1)
        np.testing.assert_array_equal(ra.accept_len, rb.accept_len)
    finally:
        a.close()
        b.close()


def test_bf16_dv_layout_runs_on_cuda_cores():
    # V = 999: the rows of a [d, V] matrix are then not 16-byte aligned, which TMA needs
    cfg = gen.Config("dv", B=2, K=5, d=128, d_draft=64, V=999, sigma_w=0.05, seed=5)
    _full_parity(cfg, (0.5,), layout=1, expect_path="simt")


@pytest.mark.parametrize("shape", [("ne_small", 3, 9, 256, 128, 3000), ("ne_pair", 6, 50, 128, 64, 1500), ("ne_k1", 5, 1, 64, 0, 300)],
                         ids=lambda s: s[0])
def test_without_the_extra_row(shape):
    """AJ_FLAG_NO_EXTRA_ROW: K rows per sequence, a last-position mismatch is rejected without the judge."""
    import paper_2504_20039_b200 as aj

    orc = _oracle()
    name, B, K, d, dd, V = shape
    cfg = gen.Config(name, B=B, K=K, d=d, d_draft=dd, V=V, sigma_W=0.2, sigma_w=0.05, match_lo=0.6, match_hi=0.95, seed=13)
    W, ht, hd, w = _host_case(cfg)
    ht = ht[:, :K].copy()
    hd = None if hd is None else hd[:, :K].copy()
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(B)])  # [B, K]
    tok = gen.plant_draft_tokens(cfg, np.concatenate([y, y[:, :1]], axis=1))
    tok[0, K - 1] = (y[0, K - 1] + 1) % V   # a sure mismatch at the last position
    tok[1, :] = y[1, :K]                    # and a sequence that passes everywhere
    case = DeviceCase(cfg, W, ht, hd, w, flags=aj.AJ_FLAG_NO_EXTRA_ROW)
    try:
        for tau in (0.0, 0.5, 1.0):
            o = orc.verify(ht, hd, W, tok, w, cfg.judge_b, tau, cfg.dtype, extra_row=False)
            g = case.run(tok, tau)
            assert g.target_tok.shape == (B, K) and g.launches == 2
            check_parity(o, g, tok, tau)
            assert np.isnan(g.judge_p[:, K - 1]).all()
            assert g.accept_len[1] == K and g.next_tok[1] == -1
            assert g.accept_len[0] <= K - 1
    finally:
        case.close()


# -------------------------------------------------------------------------------- edge cases


def test_ties_zeros_and_out_of_range_draft_tokens():
    orc = _oracle()
    cfg = gen.Config("ties", B=2, K=6, d=128, d_draft=64, V=600, sigma_w=0.05, seed=6)
    W, ht, hd, w = _host_case(cfg)
    W = W.copy()
    # duplicate rows of W: the winner of every row also appears at a higher and a lower index
    y0 = _oracle_y(cfg, W, ht)
    for v in np.unique(y0):
        if v + 37 < cfg.V:
            W[v + 37] = W[v]
    y = _oracle_y(cfg, W, ht)
    tok = gen.plant_draft_tokens(cfg, y)
    tok[0, 1] = -5          # ids outside the vocabulary are data: they simply never match
    tok[1, 2] = cfg.V + 9
    for flags in (0, 8, 1):
        case = DeviceCase(cfg, W, ht, hd, w, flags=flags)
        try:
            o = orc.verify(ht, hd, W, tok, w, 0.0, 0.5, cfg.dtype)
            g = case.run(tok, 0.5)
            np.testing.assert_array_equal(g.target_tok, o.target_tok)  # exact: ties go to the lowest index
            np.testing.assert_array_equal(g.accept_len, o.accept_len)
            np.testing.assert_array_equal(g.next_tok, o.next_tok)
        finally:
            case.close()
    # all-zero W: every logit ties at zero, the answer is token 0 everywhere; and a mix of
    # +0 and -0 logits still ties
    Wz = np.zeros_like(W)
    hneg = ht.copy()
    for flags in (0, 1):
        case = DeviceCase(cfg, Wz, hneg, hd, w, flags=flags)
        try:
            g = case.run(np.zeros((cfg.B, cfg.K), np.int32), 0.5)
            assert (g.target_tok == 0).all() and (g.accept_len == cfg.K).all() and (g.next_tok == 0).all()
            assert (g.top1 == 0).all()
        finally:
            case.close()


def test_two_sm_kernel_ties_within_and_across_the_pair():
    # More than 128 rows selects the two-SM kernel.  The winner of every row is duplicated 37 entries
    # later (same warp or the next one) and 128 entries later (the other SM of the pair, or the next
    # tile): the lowest index must win whichever SM, warp or tile sees the copy first.
    orc = _oracle()
    cfg = gen.Config("pair_ties", B=3, K=50, d=128, d_draft=64, V=900, sigma_w=0.05, seed=12)
    W, ht, hd, w = _host_case(cfg)
    W = W.copy()
    y0 = _oracle_y(cfg, W, ht)
    for v in np.unique(y0):
        for off in (37, 128):
            if v + off < cfg.V:
                W[v + off] = W[v]
    y = _oracle_y(cfg, W, ht)
    tok = gen.plant_draft_tokens(cfg, y)
    o = orc.verify(ht, hd, W, tok, w, 0.0, 0.5, cfg.dtype)
    assert (o.gap == 0).sum() >= cfg.M // 2  # most rows really are tied
    for flags in (0, 8):
        case = DeviceCase(cfg, W, ht, hd, w, flags=flags)
        try:
            g = case.run(tok, 0.5)
            assert g.path == ("umma_pair_256x256" if flags == 0 else "umma_vm_128x256")
            np.testing.assert_array_equal(g.target_tok, o.target_tok)
            np.testing.assert_array_equal(g.accept_len, o.accept_len)
            np.testing.assert_array_equal(g.next_tok, o.next_tok)
        finally:
            case.close()
    case = DeviceCase(cfg, np.zeros_like(W), ht, hd, w)
    try:
        g = case.run(np.zeros((cfg.B, cfg.K), np.int32), 0.5)
        assert (g.target_tok == 0).all() and (g.accept_len == cfg.K).all() and (g.top1 == 0).all()
    finally:
        case.close()


def test_all_negative_logits_are_not_beaten_by_the_zero_filled_tail():
    # V = 300 leaves 212 zero-filled columns in the last 256-wide (or 128-wide) tile; make every
    # real logit negative so that an unmasked tail (logit 0) would win.
    orc = _oracle()
    cfg = gen.Config("neg", B=3, K=50, d=64, d_draft=0, V=300, seed=8)
    ht = gen.f32_to_bf16_bits(np.abs(gen.bf16_bits_to_f32(gen.make_hidden(cfg)[0])))
    W = gen.f32_to_bf16_bits(-np.abs(gen.bf16_bits_to_f32(gen.make_W(cfg))))
    w = gen.make_judge(cfg)
    y = _oracle_y(cfg, W, ht)
    tok = gen.plant_draft_tokens(cfg, y)
    o = orc.verify(ht, None, W, tok, w, 0.0, 0.5, cfg.dtype)
    for flags in (0, 8):  # M = 153: two-SM kernel, one-SM kernel
        case = DeviceCase(cfg, W, ht, None, w, flags=flags)
        try:
            g = case.run(tok, 0.5)
            assert (g.top1 < 0).all()
            check_parity(o, g, tok, 0.5)
        finally:
            case.close()


def test_smallest_window_and_batch_slicing_and_determinism():
    orc = _oracle()
    cfg = gen.Config("slice", B=6, K=12, d=256, d_draft=128, V=4000, sigma_w=0.05, match_lo=0.5, match_hi=0.9, seed=9)
    W, ht, hd, w = _host_case(cfg)
    y = _oracle_y(cfg, W, ht)
    tok = gen.plant_draft_tokens(cfg, y)
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        full = case.run(tok, 0.5)
        again = case.run(tok, 0.5, fill=999)
        for a, b in zip((full.accept_len, full.next_tok, full.target_tok, full.top1), (again.accept_len, again.next_tok, again.target_tok, again.top1)):
            np.testing.assert_array_equal(a, b)  # bit-identical from run to run
        np.testing.assert_array_equal(np.isnan(full.judge_p), np.isnan(again.judge_p))
        for b in range(cfg.B):  # every sequence alone gives what it gave in the batch
            one = case.run(tok[b : b + 1], 0.5, seqs=slice(b, b + 1))
            assert one.accept_len[0] == full.accept_len[b] and one.next_tok[0] == full.next_tok[b]
            np.testing.assert_array_equal(one.target_tok[0], full.target_tok[b])
            np.testing.assert_array_equal(one.top1[0], full.top1[b])  # no split over k: bit-identical logits
        # K = 1 on the first two rows of each sequence
        ht1, hd1 = ht[:, :2].copy(), hd[:, :2].copy()
        cfg1 = gen.scaled(cfg, K=1)
        c1 = DeviceCase(cfg1, case.W, ht1, hd1, w)
        try:
            o = orc.verify(ht1, hd1, W, tok[:, :1], w, 0.0, 0.5, cfg.dtype)
            check_parity(o, c1.run(tok[:, :1], 0.5), tok[:, :1], 0.5)
        finally:
            c1.close()
    finally:
        case.close()


def test_error_paths_enqueue_nothing():
    import torch

    import paper_2504_20039_b200 as aj

    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 0, 4, 256, 128, 1000)
    assert e.value.status == aj.AJ_ERR_INVALID_ARG
    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 1, 4, 100, 128, 1000)  # bf16 needs d % 8 == 0
    assert e.value.status == aj.AJ_ERR_UNSUPPORTED
    with pytest.raises(aj.AjError) as e:
        aj.Handle(99, 1, 4, 256, 128, 1000)
    assert e.value.status == aj.AJ_ERR_CUDA
    cfg = gen.Config("err", B=2, K=4, d=128, d_draft=64, V=500, seed=1)
    W, ht, hd, w = _host_case(cfg)
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        i32 = dict(dtype=torch.int32, device="cuda")
        tok = torch.zeros((2, 4), **i32)
        acc = torch.full((2,), -1, **i32)
        nxt = torch.full((2,), -1, **i32)
        h = case.handle
        args = dict(accept_len=acc, next_tok=nxt, check=False)
        assert h.verify(None, case.hd, case.W, tok, case.w, 0.0, 0.5, 2, 4, **args) == aj.AJ_ERR_INVALID_ARG
        assert h.verify(case.ht, None, case.W, tok, case.w, 0.0, 0.5, 2, 4, **args) == aj.AJ_ERR_INVALID_ARG
        assert h.verify(case.ht, case.hd, case.W, tok, case.w, 0.0, 0.5, 0, 4, **args) == aj.AJ_ERR_INVALID_ARG
        assert h.verify(case.ht, case.hd, case.W, tok, case.w, 0.0, 0.5, 3, 4, **args) == aj.AJ_ERR_WORKSPACE
        assert h.verify(case.ht, case.hd, case.W, tok, case.w, 0.0, 0.5, 2, 5, **args) == aj.AJ_ERR_WORKSPACE
        assert h.verify(case.ht, case.hd, case.W, tok, case.w, 0.0, 0.5, 2, 4, accept_len=None, next_tok=nxt, check=False) == aj.AJ_ERR_INVALID_ARG
        misaligned = case.ht.view(torch.int16).flatten()[1:]  # 2 bytes off a 16-byte boundary
        assert h.verify(misaligned, case.hd, case.W, tok, case.w, 0.0, 0.5, 1, 4, **args) == aj.AJ_ERR_UNSUPPORTED
        torch.cuda.synchronize()
        assert (acc.cpu() == -1).all() and (nxt.cpu() == -1).all()
        assert h.last_status() == aj.AJ_OK
    finally:
        case.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    import torch

    cfg = gen.Config("host", B=4, K=20, d=512, d_draft=256, V=9000, sigma_w=0.05, match_lo=0.5, match_hi=0.9, seed=10)
    W, ht, hd, w = _host_case(cfg)
    y = _oracle_y(cfg, W, ht)
    tok = gen.plant_draft_tokens(cfg, y)
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        g = case.run(tok, 0.5)
        pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
        ht_h, hd_h, tok_h = pin(ht), pin(hd), pin(tok)
        acc = torch.full((cfg.B,), -1, dtype=torch.int32).pin_memory()
        nxt = torch.full((cfg.B,), -1, dtype=torch.int32).pin_memory()
        tt = torch.full((cfg.B, cfg.K + 1), -1, dtype=torch.int32).pin_memory()
        case.handle.verify_host(ht_h, hd_h, case.W, tok_h, case.w, 0.0, 0.5, cfg.B, cfg.K, acc, nxt, tt,
                                stream=torch.cuda.current_stream().cuda_stream)
        np.testing.assert_array_equal(acc.numpy(), g.accept_len)
        np.testing.assert_array_equal(nxt.numpy(), g.next_tok)
        np.testing.assert_array_equal(tt.numpy(), g.target_tok)
        # pageable host buffers (plain numpy arrays) take the copying route and give the same
        acc2, nxt2, tt2 = np.full(cfg.B, -1, np.int32), np.full(cfg.B, -1, np.int32), np.full((cfg.B, cfg.K + 1), -1, np.int32)
        case.handle.verify_host(ht.copy(), hd.copy(), case.W, tok.copy(), case.w, 0.0, 0.5, cfg.B, cfg.K, acc2, nxt2, tt2,
                                stream=torch.cuda.current_stream().cuda_stream)
        np.testing.assert_array_equal(acc2, g.accept_len)
        np.testing.assert_array_equal(nxt2, g.next_tok)
        np.testing.assert_array_equal(tt2, g.target_tok)
    finally:
        case.close()


def test_host_entry_point_reads_the_host_buffers_afresh_every_cycle():
    """The same pinned buffers are rewritten by the host between cycles (a small batch is fetched from them by
    a kernel, a large one by the copy engines): every cycle must see what they hold then.  Also the
    target-only classifier, where there is no second tensor to fetch."""
    import torch

    orc = _oracle()
    for name, B, K, d, dd, V in (("host_small", 4, 20, 512, 256, 9000), ("host_target_only", 3, 12, 256, 0, 4000),
                                 ("host_large", 24, 40, 768, 256, 3000)):  # 24 x 41 x (768 + 256) x 2 B = 2 MB: copy engines
        cfg = gen.Config(name, B=B, K=K, d=d, d_draft=dd, V=V, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.9, seed=19)
        W, ht, hd, w = _host_case(cfg)
        tok = gen.plant_draft_tokens(cfg, _oracle_y(cfg, W, ht))
        case = DeviceCase(cfg, W, ht, hd, w)
        try:
            pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
            ht_h, tok_h = pin(ht.copy()), pin(tok.copy())
            hd_h = pin(hd.copy()) if dd else None
            acc = torch.full((cfg.B,), -1, dtype=torch.int32).pin_memory()
            nxt = torch.full((cfg.B,), -1, dtype=torch.int32).pin_memory()
            tt = torch.full((cfg.B, cfg.K + 1), -1, dtype=torch.int32).pin_memory()
            order = np.arange(cfg.B)
            for cycle in range(4):
                # rotate the sequences through the same buffers, in place
                order = np.roll(order, 1)
                ht_h.numpy()[:] = ht[order].view(np.int16)
                tok_h.numpy()[:] = tok[order]
                if dd:
                    hd_h.numpy()[:] = hd[order].view(np.int16)
                case.handle.verify_host(ht_h, hd_h, case.W, tok_h, case.w, cfg.judge_b, 0.5, cfg.B, cfg.K, acc, nxt, tt,
                                        stream=torch.cuda.current_stream().cuda_stream)
                o = orc.verify(ht[order], hd[order] if dd else None, W, tok[order], w, cfg.judge_b, 0.5, cfg.dtype)
                np.testing.assert_array_equal(tt.numpy(), o.target_tok)
                np.testing.assert_array_equal(acc.numpy(), o.accept_len)
                np.testing.assert_array_equal(nxt.numpy(), o.next_tok)
        finally:
            case.close()


def test_a_cycle_captured_in_a_cuda_graph_replays_with_new_inputs():
    """aj_verify only enqueues (two kernel launches, no allocation, no synchronisation), so a cycle can be
    captured in a CUDA graph and replayed: the replay reads whatever the input buffers hold then."""
    import torch

    orc = _oracle()
    cfg = gen.Config("graph", B=3, K=12, d=256, d_draft=128, V=4000, sigma_W=0.2, sigma_w=0.05, match_lo=0.5, match_hi=0.9, seed=14)
    W, ht, hd, w = _host_case(cfg)
    y = _oracle_y(cfg, W, ht)
    tok = gen.plant_draft_tokens(cfg, y)
    case = DeviceCase(cfg, W, ht, hd, w)
    try:
        case.run(tok, 0.5)  # warms the handle up (tensor maps cached) before the capture
        i32 = dict(dtype=torch.int32, device="cuda")
        tok_d = torch.zeros((cfg.B, cfg.K), **i32)
        acc, nxt, tt = torch.zeros(cfg.B, **i32), torch.zeros(cfg.B, **i32), torch.zeros((cfg.B, cfg.K + 1), **i32)
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                case.handle.verify(case.ht, case.hd, case.W, tok_d, case.w, cfg.judge_b, 0.5, cfg.B, cfg.K, acc, nxt, tt,
                                   stream=torch.cuda.current_stream().cuda_stream)
        torch.cuda.current_stream().wait_stream(side)
        for trial in range(3):
            cur = tok if trial != 1 else np.roll(tok, 1, axis=1)  # other draft tokens on the second replay
            tok_d.copy_(torch.from_numpy(np.ascontiguousarray(cur)))
            graph.replay()
            torch.cuda.synchronize()
            got = (tt.cpu().numpy(), acc.cpu().numpy(), nxt.cpu().numpy())
            direct = case.run(cur, 0.5)  # the same cycle enqueued directly
            np.testing.assert_array_equal(got[0], direct.target_tok)
            np.testing.assert_array_equal(got[1], direct.accept_len)
            np.testing.assert_array_equal(got[2], direct.next_tok)
            check_parity(orc.verify(ht, hd, W, cur, w, cfg.judge_b, 0.5, cfg.dtype), direct, cur, 0.5)
        assert case.handle.last_status() == case.aj.AJ_OK
    finally:
        case.close()
