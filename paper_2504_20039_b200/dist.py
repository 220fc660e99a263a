"""Process-group plumbing for running the verify-and-judge step on several GPUs of one node.

One process per GPU.  Sequences are independent (each is verified against the whole LM head), so the
batch-parallel form needs no data-path collective: every rank verifies its own batch against its own
copy of W_lm, and the process group only serves the barrier and the max-over-ranks of the timings.
torch.distributed is used for exactly that; on a machine without GPUs the same code runs over gloo.
"""
from __future__ import annotations

import os
from dataclasses import dataclass, replace


@dataclass(frozen=True)
class RankInfo:
    rank: int
    world: int
    local_rank: int


def rank_info() -> RankInfo:
    """Rank layout from the launcher's environment (torchrun / torch.distributed.run)."""
    return RankInfo(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                    int(os.environ.get("LOCAL_RANK", "0")))


def rank_config(cfg, rank: int):
    """The batch rank `rank` verifies: the same shape as cfg, its own seeded sequences.

    Rank 0 keeps cfg's seed, so a one-rank job is exactly the single-GPU workload."""
    return cfg if rank == 0 else replace(cfg, seed=cfg.seed + 7919 * rank)


def sampling_seed(seed: int, rank: int, sharding: str = "batch") -> int:
    """The seed rank `rank` gives aj_set_sampling.  Ranks that verify different sequences (batch sharding) must
    draw different noise, and every handle numbers its rows from zero, so each gets its own seed; the ranks of
    a vocabulary-parallel group verify the same rows and must all use the same one."""
    if sharding == "vocab":
        return seed & (2**64 - 1)
    return (seed + 0x9E3779B97F4A7C15 * rank) & (2**64 - 1)


def job_positions(cfg, world: int) -> int:
    """Draft positions the whole job verifies per step: every rank's B*K."""
    return cfg.B * cfg.K * world


def split_sequences(total: int, world: int):
    """Contiguous, near-equal shares of `total` sequences: [(start, count)] per rank; every sequence
    lands on exactly one rank.  Used when a fixed global batch is divided over the ranks."""
    base, rem = divmod(total, world)
    out, start = [], 0
    for r in range(world):
        n = base + (1 if r < rem else 0)
        out.append((start, n))
        start += n
    return out


class Exchange:
    """The exchange buffers of a vocabulary-parallel group, one per rank, as addressable from this
    process: the own buffer is allocated here, the peers' are mapped through CUDA IPC handles that the
    ranks swap over the process group.  `buffers[r]` is rank r's; pass the list to Handle(shard=...)."""

    def __init__(self, group: "Group", max_B: int, max_K: int):
        """Fails on EVERY rank if it fails on one (a rank that raised alone would leave the others waiting at
        the next barrier): after each step the ranks vote, and a rank that succeeded undoes its part."""
        from . import binding as aj

        self._aj, self.group = aj, group
        rank, world = group.info.rank, group.info.world
        self.own, self.buffers, err, handle = None, [], None, b""
        try:
            self.own = aj.shard_exchange_alloc(max_B, max_K, world)
            handle = aj.ipc_export(self.own)
        except Exception as e:  # noqa: BLE001 - reported to every rank below
            err = e
        handles = group.all_gather_bytes(handle)
        if not group.all_ok(err is None):
            self._undo()
            raise RuntimeError(f"exchange buffer could not be allocated or exported on some rank (this rank: {err!r})")
        try:
            self.buffers = [self.own if r == rank else aj.ipc_import(handles[r]) for r in range(world)]
        except Exception as e:  # noqa: BLE001
            err = e
        if not group.all_ok(err is None):  # also: every rank has mapped every buffer
            self._undo()
            raise RuntimeError(f"a peer's exchange buffer could not be mapped on some rank (this rank: {err!r})")

    def _undo(self) -> None:
        for r, p in enumerate(self.buffers):
            if r != self.group.info.rank and p:
                try:
                    self._aj.ipc_close(p)
                except Exception:  # noqa: BLE001
                    pass
        self.buffers = []
        if self.own:
            try:
                self._aj.shard_exchange_free(self.own)
            except Exception:  # noqa: BLE001
                pass
            self.own = None

    def ready(self) -> None:
        """Call after every rank has created its handle (which clears its own buffer) and before the first cycle."""
        self.group.barrier()

    def close(self) -> None:
        """Call after the last cycle has finished on this rank's stream."""
        self.group.barrier()  # no rank is still publishing into a buffer about to go away
        for r, p in enumerate(self.buffers):
            if r != self.group.info.rank:
                self._aj.ipc_close(p)
        self.group.barrier()
        self._aj.shard_exchange_free(self.own)
        self.buffers = []


class Group:
    """A thin wrapper over torch.distributed that degrades to a no-op for a single process."""

    def __init__(self, info: RankInfo | None = None, backend: str | None = None, device=None):
        self.info = info or rank_info()
        self.device = device
        self.dist = None
        self.backend = backend
        if self.info.world > 1:
            import torch
            import torch.distributed as dist

            if backend is None:
                backend = "nccl" if torch.cuda.is_available() else "gloo"
            kw = {}
            if backend == "nccl" and device is not None:
                kw["device_id"] = device
            if not dist.is_initialized():
                dist.init_process_group(backend, rank=self.info.rank, world_size=self.info.world, **kw)
            self.dist = dist
            self.backend = backend

    def _reduce(self, x: float, op_name: str) -> float:
        if self.dist is None:
            return float(x)
        import torch

        dev = self.device if (self.backend == "nccl" and self.device is not None) else "cpu"
        t = torch.tensor([float(x)], dtype=torch.float64, device=dev)
        self.dist.all_reduce(t, op=getattr(self.dist.ReduceOp, op_name))
        return float(t.item())

    def barrier(self) -> None:
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, x: float) -> float:
        """The slowest rank's value: multi-GPU timings are reported as the max over ranks."""
        return self._reduce(x, "MAX")

    def sum_over_ranks(self, x: float) -> float:
        return self._reduce(x, "SUM")

    def all_ok(self, ok: bool) -> bool:
        """True iff `ok` is true on every rank (a collective: all ranks get the same answer)."""
        return self._reduce(1.0 if ok else 0.0, "MIN") > 0.5

    def all_gather_bytes(self, payload: bytes):
        """Every rank's `payload`, in rank order (used to exchange IPC handles of exchange buffers)."""
        if self.dist is None:
            return [bytes(payload)]
        out = [None] * self.info.world
        self.dist.all_gather_object(out, bytes(payload))
        return out

    def close(self) -> None:
        if self.dist is not None and self.dist.is_initialized():
            self.dist.destroy_process_group()
            self.dist = None
