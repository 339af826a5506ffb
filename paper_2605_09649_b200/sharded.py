"""Eviction round of sequences whose layers are sharded over ranks (one global budget over all layers and heads,
Sec. 4.2 of the paper): the exchange protocol around the library's rank-local stages (trimkv_shard_* in include/trimkv.h).

Every rank holds the pools of a slice of the layers.  The selection is the single-GPU one (key sample -> bracket of the
threshold -> one filter pass -> exact ranking of the keys inside the bracket) with three small exchanges:

    all-gather   sample keys            <= 4096 keys x 8 B per sequence and rank (about 3072 keys over all ranks)
    all-reduce   counts below bracket   8 B per sequence            (+ all-gather of the candidate counts, 4 B)
    all-gather   candidate records      16 B each; a few thousand per sequence in a decode step

After each exchange every rank computes the same thing from the same data, so all ranks reach the same threshold and
each flags its own entries.  If the bracket missed (or a list overflowed) every rank sees it, and an exact radix select
runs instead: six rounds of a local 2048-bin histogram and an all-reduce (8 KB per sequence and round).

This module holds no arithmetic of the method: `stages` does the rank-local work (CudaStages: the CUDA kernels through
the C ABI), `comm` moves tensors (TorchComm: torch.distributed, i.e. NCCL between GPUs).
"""
from __future__ import annotations

import ctypes as C
from typing import List

import torch

from . import binding

DIGIT_BITS = 11                    # digit of the exact fallback's radix select (2048 bins)


class TorchComm:
    """Collectives over a torch.distributed process group (NCCL for CUDA tensors, gloo for CPU tensors)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        """[world, *t.shape], in rank order."""
        out = torch.empty((self.world,) + tuple(t.shape), dtype=t.dtype, device=t.device)
        self.dist.all_gather_into_tensor(out.view(-1), t.contiguous().view(-1), group=self.group)
        return out

    def all_reduce_sum(self, t: torch.Tensor) -> torch.Tensor:
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)
        return t


class CudaStages:
    """Rank-local stages on a handle created with shard_total_layers > 0 (argument marshalling only)."""

    def __init__(self, cache: "binding.TrimKV"):
        self.cache, self.B = cache, cache.B
        self.dev = torch.device("cuda", torch.cuda.current_device())
        self.sample_cap = int(binding.lib().trimkv_shard_sample_cap())

    def _call(self, name, *args):
        binding._check(getattr(binding.lib(), name)(self.cache._h, *args, binding._stream()))

    def sample(self, n_total, k_evict):
        keys = torch.empty(self.B, self.sample_cap, dtype=torch.int64, device=self.dev)
        counts = torch.empty(self.B, dtype=torch.int32, device=self.dev)
        self._call("trimkv_shard_sample", n_total, k_evict, binding._ptr(keys), binding._ptr(counts))
        return keys, counts

    def bracket(self, gkeys, gcounts, n_total, k_evict):
        self._call("trimkv_shard_bracket", gkeys.shape[0], binding._ptr(gkeys), binding._ptr(gcounts), n_total, k_evict)

    def filter(self):
        n_below = torch.empty(self.B, dtype=torch.int64, device=self.dev)
        cand_count = torch.empty(self.B, dtype=torch.int32, device=self.dev)
        self._call("trimkv_shard_filter", binding._ptr(n_below), binding._ptr(cand_count))
        return n_below, cand_count

    def candidates(self, cap):
        out = torch.zeros(self.B, cap, 2, dtype=torch.int64, device=self.dev)         # records {key, slot}
        self._call("trimkv_shard_candidates", cap, binding._ptr(out))
        return out

    def resolve(self, gcand, gcounts, n_below_global, k_evict, cap, rank):
        resolved = torch.empty(self.B, dtype=torch.int32, device=self.dev)
        self._call("trimkv_shard_resolve", gcand.shape[0], rank, cap, binding._ptr(gcand), binding._ptr(gcounts),
                   binding._ptr(n_below_global), k_evict, binding._ptr(resolved))
        return resolved

    def new_prefix_rank(self, k_evict):
        return (torch.zeros(self.B, dtype=torch.int64, device=self.dev),
                torch.full((self.B,), k_evict, dtype=torch.int64, device=self.dev))

    def hist(self, prefix, top):
        out = torch.empty(self.B, 1 << DIGIT_BITS, dtype=torch.int32, device=self.dev)
        self._call("trimkv_shard_hist", binding._ptr(prefix), top, binding._ptr(out))
        return out

    def digit(self, hist, prefix, rank, top):
        self._call("trimkv_shard_digit", binding._ptr(hist), binding._ptr(prefix), binding._ptr(rank), top)

    def mark(self, tau):
        self._call("trimkv_shard_mark", binding._ptr(tau))

    def compact(self) -> List[int]:
        out = (C.c_int64 * self.B)()
        self._call("trimkv_shard_compact", out)
        return list(out)


def sharded_evict(stages, comm, n_total: int, k_evict: int) -> dict:
    """One eviction round: evict the k_evict lowest-scoring of the n_total entries that every sequence holds over ALL
    ranks.  Every rank calls this with the same numbers.  Returns what happened (for tests and tuning)."""
    keys, counts = stages.sample(n_total, k_evict)
    gkeys, gcounts = comm.all_gather(keys), comm.all_gather(counts)
    stages.bracket(gkeys, gcounts, n_total, k_evict)
    n_below, cand_count = stages.filter()
    comm.all_reduce_sum(n_below)
    gcc = comm.all_gather(cand_count)                            # [world, B]; -1 where a rank's list overflowed
    cap = max(int(gcc.max().item()), 1)                          # the one host read-back of the normal path
    gcand = comm.all_gather(stages.candidates(cap))
    resolved = stages.resolve(gcand, gcc, n_below, k_evict, cap, comm.rank)
    info = {"candidates": int(gcc.clamp(min=0).sum().item()), "exchange_bytes": int(gkeys.numel() * 8 + gcand.numel() * 8),
            "fallback": False}
    if not bool(resolved.bool().all().item()):                   # same flags on every rank: all take the fallback together
        info["fallback"] = True
        prefix, rank = stages.new_prefix_rank(k_evict)
        top = 64
        while top > 0:
            h = stages.hist(prefix, top)
            comm.all_reduce_sum(h)
            stages.digit(h, prefix, rank, top)
            top -= min(DIGIT_BITS, top)
        stages.mark(prefix)
    info["local_entries"] = stages.compact()
    return info
