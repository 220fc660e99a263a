"""The C-ABI library loads without a GPU and exports every symbol include/aj_verify.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_2504_20039_b200 import build as b

    return b.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "aj_verify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aj_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(built):
    lib = ctypes.CDLL(built)
    names = _declared()
    assert {"aj_create", "aj_verify", "aj_verify_host", "aj_destroy", "aj_last_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_the_header(built):
    import paper_2504_20039_b200 as aj
    from paper_2504_20039_b200 import binding

    aj.lib()
    assert sorted(binding.EXPORTS) == _declared()
    assert "sm_100a" in aj.version()
    assert aj.status_string(aj.AJ_ERR_TIMEOUT)


def test_argument_checks_need_no_device(built):
    import torch

    import paper_2504_20039_b200 as aj

    for args in [(0, 0, 4, 256, 128, 1000), (0, 1, 0, 256, 128, 1000), (0, 1, 2000, 256, 128, 1000),
                 (0, 1, 4, 0, 128, 1000), (0, 1, 4, 256, -1, 1000), (0, 1, 4, 256, 128, 0), (-1, 1, 4, 256, 128, 1000)]:
        with pytest.raises(aj.AjError) as e:
            aj.Handle(*args)
        assert e.value.status == aj.AJ_ERR_INVALID_ARG, args
    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 1, 4, 250, 128, 1000, aj.AJ_BF16)
    assert e.value.status == aj.AJ_ERR_UNSUPPORTED
    with pytest.raises(aj.AjError) as e:
        aj.Handle(0, 1, 4, 256, 128, 1000, 7)
    assert e.value.status == aj.AJ_ERR_INVALID_ARG
    if not torch.cuda.is_available():  # no device: creation fails cleanly, there is no CPU fallback
        with pytest.raises(aj.AjError) as e:
            aj.Handle(0, 1, 4, 256, 128, 1000)
        assert e.value.status == aj.AJ_ERR_CUDA


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2504_20039_b200 import binding

    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        binding.lib()


def test_two_sm_schedule_covers_every_row_once(built):
    """Host arithmetic of the two-SM kernel's tiling: tiles of at most 256 rows in units of 16 that
    cover the batch exactly once with no padded tile, and groups that cover every tile once."""
    import paper_2504_20039_b200 as aj

    for M, d in [(129, 4096), (136, 4096), (256, 4096), (257, 4096), (264, 4096), (500, 4096), (512, 4096), (513, 4096),
                 (520, 4096), (2112, 4096), (2080, 8192), (8448, 4096), (16640, 4096), (16640, 8192), (4097, 64)]:
        s = aj.pair_schedule(M, d, 128256)
        assert s["n_v"] == 501
        units = (M + 15) // 16
        assert s["dual"] == (1 if M > 256 else 0)              # wide tiles (two accumulators) above 256 rows
        cap = 32 if s["dual"] else 16                         # units per tile: two accumulators or one
        sizes = [s["u_base"] + (i < s["u_rem"]) for i in range(s["n_n"])]
        assert sum(sizes) == units and max(sizes) <= cap and min(sizes) >= (2 if s["dual"] else 1)
        assert s["n_n"] == -(-units // cap)                   # the fewest tiles
        assert max(sizes) - min(sizes) <= 1                   # spread evenly
        per_acc = -(-max(sizes) // 2) if s["dual"] else max(sizes)
        assert s["box_rows"] == 8 * per_acc <= 128
        # a stage holds two k-blocks of 64 where three such stages fit in the ring (and d / 64 is even), else one
        sub = 16384 + (2 if s["dual"] else 1) * s["box_rows"] * 128
        kps = 2 if ((d // 64) % 2 == 0 and (224 * 1024) // (2 * sub) >= 3) else 1
        stage = kps * sub
        assert 3 <= s["stages"] == min(8, (224 * 1024) // stage) and s["stages"] * stage <= 224 * 1024
        groups = [s["g_base"] + (g < s["g_rem"]) for g in range(s["n_groups"])]
        assert sum(groups) == s["n_n"] and min(groups) >= 1 and max(groups) - min(groups) <= 1
        assert max(groups) * (512 if s["dual"] else 256) * d * 2 <= 40 << 20 or max(groups) == 1
    assert aj.pair_schedule(2112, 4096, 128256)["n_groups"] == 1
    assert aj.pair_schedule(2080, 8192, 128256)["n_groups"] == 1
    assert aj.pair_schedule(16640, 4096, 128256)["n_groups"] == 4


def test_shard_ranges_are_whole_blocks_that_cover_the_vocabulary(built):
    import paper_2504_20039_b200 as aj

    for V in (128256, 1000, 256, 255, 70001):
        for world in range(1, 9):
            if -(-V // 256) < world:  # fewer blocks than GPUs: refused, no GPU gets an empty shard
                with pytest.raises(aj.AjError):
                    aj.shard_range(V, world, 0)
                continue
            parts = [aj.shard_range(V, world, r) for r in range(world)]
            assert min(n for _, n in parts) >= 1
            assert parts[0][0] == 0 and sum(n for _, n in parts) == V
            for (b0, n0), (b1, _) in zip(parts, parts[1:]):
                assert b0 + n0 == b1
            assert all(b % 256 == 0 for b, _ in parts)
            blocks = [-(-n // 256) for _, n in parts]
            assert max(blocks) - min(blocks) <= 1
    assert aj.shard_range(128256, 8, 0) == (0, 63 * 256) and aj.shard_range(128256, 8, 7) == (128256 - 62 * 256, 62 * 256)
    assert aj.shard_exchange_bytes(4, 8, 9) == 0 and aj.shard_exchange_bytes(4, 8, 2) == 256 + 2 * 2 * 36 * 8
    with pytest.raises(aj.AjError):
        aj.shard_range(1000, 9, 0)
    with pytest.raises(aj.AjError):
        aj.shard_range(1000, 2, 2)
