"""Sharing an exchange buffer between two processes of one node through aj_ipc_export / aj_ipc_import.

Both processes use the same GPU here.  Only the importing process launches kernels (a vocabulary-parallel
group of one whose exchange buffer is the memory the other process allocated), so no kernel ever waits
for another process."""
import numpy as np
import pytest

import aj_inputs as gen

pytestmark = pytest.mark.gpu


def _importer(handle_bytes, out):
    try:
        import torch

        import paper_2504_20039_b200 as aj
        from aj_testlib import DeviceCase

        torch.cuda.set_device(0)
        cfg = gen.Config("ipc", B=2, K=6, d=128, d_draft=64, V=1500, sigma_W=0.2, sigma_w=0.05, seed=40)
        W, (ht, hd), w = gen.make_W(cfg), gen.make_hidden(cfg), gen.make_judge(cfg)
        tok = gen.random_draft_tokens(cfg)
        case = DeviceCase(cfg, W, ht, hd, w)
        ptr = aj.ipc_import(handle_bytes)
        h = aj.Handle(0, cfg.B, cfg.K, cfg.d, cfg.d_draft, cfg.V, cfg.dtype, aj.AJ_W_VD, 0, shard=(0, 1, 0, cfg.V, [ptr]))
        try:
            want = case.run(tok, 0.5)
            i32 = dict(dtype=torch.int32, device="cuda")
            acc, nxt, tt = torch.zeros(cfg.B, **i32), torch.zeros(cfg.B, **i32), torch.zeros((cfg.B, cfg.K + 1), **i32)
            for _ in range(2):
                h.verify(case.ht, case.hd, case.W, torch.from_numpy(tok).cuda(), case.w, cfg.judge_b, 0.5, cfg.B, cfg.K, acc, nxt, tt)
            torch.cuda.synchronize()
            ok = (h.last_status() == aj.AJ_OK and (tt.cpu().numpy() == want.target_tok).all()
                  and (acc.cpu().numpy() == want.accept_len).all() and (nxt.cpu().numpy() == want.next_tok).all())
        finally:
            h.destroy()
            case.close()
            aj.ipc_close(ptr)
        out.put("ok" if ok else "mismatch")
    except Exception as e:  # pragma: no cover
        out.put(f"error: {e!r}")


def test_exported_buffer_serves_as_exchange_buffer_in_another_process():
    import torch
    import torch.multiprocessing as mp

    import paper_2504_20039_b200 as aj

    torch.cuda.set_device(0)
    own = aj.shard_exchange_alloc(2, 6, 1)
    try:
        handle = aj.ipc_export(own)
        assert len(handle) == 64
        ctx = mp.get_context("spawn")
        out = ctx.Queue()
        p = ctx.Process(target=_importer, args=(handle, out))
        p.start()
        msg = out.get(timeout=300)
        p.join(timeout=60)
        assert msg == "ok" and p.exitcode == 0
    finally:
        aj.shard_exchange_free(own)
    with pytest.raises(aj.AjError):
        aj.ipc_import(b"\0" * 64)  # not a handle: a clean error
