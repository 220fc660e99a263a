"""The multi-process plumbing (one process per GPU) over gloo on CPU, world size 2: rank layout,
per-rank batches, max-over-ranks timing, whole-job throughput arithmetic, handle exchange."""
import os
import socket

import pytest

import aj_inputs as gen
from paper_2504_20039_b200 import dist as ajd


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    g = ajd.Group(backend="gloo")
    try:
        assert g.info == ajd.RankInfo(rank, world, rank)
        cfg = ajd.rank_config(gen.scaled(gen.C1, B=3), rank)
        ht, _ = gen.make_hidden(cfg)
        g.barrier()
        slowest = g.max_over_ranks(10.0 + rank)          # rank r "took" 10 + r ms
        total = g.sum_over_ranks(float(cfg.B * cfg.K))    # positions verified by the whole job
        handles = g.all_gather_bytes(bytes([rank]) * 64)  # stand-ins for 64-byte IPC handles
        seeds = g.all_gather_bytes(ajd.sampling_seed(77, rank).to_bytes(8, "little"))
        assert len({bytes(s) for s in seeds}) == world and ajd.sampling_seed(77, rank, "vocab") == 77
        votes = (g.all_ok(True), g.all_ok(rank != 1))       # one rank's failure is every rank's answer
        # Exchange set-up against a fake of the CUDA calls: rank 1 cannot map rank 0's buffer; both ranks must
        # raise, and both must give back what they had allocated and mapped
        from paper_2504_20039_b200 import binding

        log = []
        binding.shard_exchange_alloc = lambda B, K, w: 1000 + rank
        binding.shard_exchange_free = lambda p: log.append(("free", p))
        binding.ipc_export = lambda p: bytes([rank]) * 64
        binding.ipc_close = lambda p: log.append(("close", p))

        def fake_import(h):
            if rank == 1:
                raise RuntimeError("peer mapping refused")
            return 2000 + h[0]

        binding.ipc_import = fake_import
        try:
            ajd.Exchange(g, 4, 8)
            raised = False
        except RuntimeError:
            raised = True
        binding.ipc_import = lambda h: 2000 + h[0]
        ex = ajd.Exchange(g, 4, 8)                            # and with every call succeeding it is built
        built = ex.buffers == ([1000, 2001] if rank == 0 else [2000, 1001])
        out.put((rank, cfg.seed, float(ht.astype("float64").sum()), slowest, total, [h[0] for h in handles], len(handles[0]),
                 votes, raised, sorted(log), built))
    finally:
        g.close()


def test_two_ranks_over_gloo():
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, sum0, slow0, tot0, hs0, n0, *more0), (r1, seed1, sum1, slow1, tot1, hs1, n1, *more1) = res
    assert more0[0] == more1[0] == (True, False)
    assert more0[1] and more1[1]                                           # the failure on rank 1 raised on both ranks
    assert more0[2] == [("close", 2001), ("free", 1000)] and more1[2] == [("free", 1001)]
    assert more0[3] and more1[3]
    assert (r0, r1) == (0, 1)
    assert seed0 == gen.C1.seed and seed1 != seed0 and sum0 != sum1      # each rank verifies its own sequences
    assert slow0 == slow1 == 11.0                                          # every rank reports the slowest rank's time
    assert tot0 == tot1 == ajd.job_positions(gen.scaled(gen.C1, B=3), 2)   # value = all ranks' positions / that time
    assert hs0 == hs1 == [0, 1] and n0 == n1 == 64                         # handles arrive in rank order on every rank


def test_single_process_group_is_a_no_op():
    g = ajd.Group(ajd.RankInfo(0, 1, 0))
    g.barrier()
    assert g.max_over_ranks(3.5) == 3.5 and g.sum_over_ranks(2.0) == 2.0
    assert g.all_gather_bytes(b"ab") == [b"ab"]
    g.close()


@pytest.mark.parametrize("total,world", [(64, 8), (7, 2), (3, 4), (256, 3)])
def test_split_sequences_covers_every_sequence_once(total, world):
    parts = ajd.split_sequences(total, world)
    assert len(parts) == world and parts[0][0] == 0
    assert sum(n for _, n in parts) == total
    assert all(parts[i][0] + parts[i][1] == parts[i + 1][0] for i in range(world - 1))
    assert max(n for _, n in parts) - min(n for _, n in parts) <= 1
