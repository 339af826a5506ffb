"""Test infrastructure for the layer-sharded eviction round (paper_2605_09649_b200/sharded.py).

HostStages is a plain numpy statement of the rank-local stages (sample, bracket, filter, exact ranking, the radix
fallback, compaction) with the interface of sharded.CudaStages, so that the exchange protocol can run on CPU ranks
(gloo) and be compared with the single-process oracle.  Scores come from the oracle's `score`; keys are the
(score, older position, lower layer, lower head) order of its `select_keep`, packed into 64 bits.
ThreadComm lets several emulated ranks run the protocol inside one process (one thread per rank).
"""
from __future__ import annotations

import threading

import numpy as np
import torch

from oracle import trimkv_oracle as orc

SAMPLE_CAP, SAMPLE_MEAN = 4096, 3072
U64 = np.uint64
ALL1 = np.uint64(0xFFFFFFFFFFFFFFFF)


def pool_bits_of(total_pools: int) -> int:
    b = 0
    while (1 << b) < total_pools:
        b += 1
    return max(1, b)


def eviction_keys(S32, pos, pool, pool_bits):
    """64-bit keys whose ascending order is the eviction order: lowest score first; among equal scores the newer
    position, then the higher pool id (layer * H + head), goes first."""
    s = (np.asarray(S32, np.float32) + np.float32(0.0)).view(np.uint32).astype(np.uint64)      # -0 folded onto +0
    neg = (s & U64(0x80000000)) != 0
    k32 = np.where(neg, (~s) & U64(0xFFFFFFFF), s | U64(0x80000000))
    tie = (np.asarray(pos, np.uint64) << U64(pool_bits)) | np.asarray(pool, np.uint64)
    return (k32 << U64(32)) | ((~tie) & U64(0xFFFFFFFF))


class HostStages:
    def __init__(self, rank, layer0, layers, total_layers, kv_heads, batch, horizon=2, distrust=False):
        self.rank, self.l0, self.L, self.Ltot, self.H, self.B = rank, layer0, layers, total_layers, kv_heads, batch
        self.horizon, self.distrust = horizon, distrust
        self.pool_bits = pool_bits_of(total_layers * kv_heads)
        self.tokens = 0
        self.round = 0
        z = lambda dt: [np.zeros(0, dt) for _ in range(batch)]
        self.pos, self.lam, self.c, self.pool = z(np.int64), z(np.float32), z(np.float32), z(np.int64)

    # ---- cache content
    def append_token_block(self, lam, c):
        """lam, c: [L_local, B, n, H] fp32 for n new tokens of every local layer."""
        n = lam.shape[2]
        newpos = self.tokens + 1 + np.arange(n, dtype=np.int64)
        for b in range(self.B):
            for l in range(self.L):
                for h in range(self.H):
                    self.pos[b] = np.concatenate([self.pos[b], newpos])
                    self.lam[b] = np.concatenate([self.lam[b], lam[l, b, :, h]])
                    self.c[b] = np.concatenate([self.c[b], c[l, b, :, h]])
                    self.pool[b] = np.concatenate([self.pool[b], np.full(n, (self.l0 + l) * self.H + h, np.int64)])
        self.tokens += n

    def kept_positions(self, b, layer_global, head):
        sel = self.pool[b] == layer_global * self.H + head
        return np.sort(self.pos[b][sel])

    def _keys(self, b):
        S = orc.score(self.lam[b], self.c[b], self.pos[b], self.tokens)
        return eviction_keys(S, self.pos[b], self.pool[b], self.pool_bits)

    # ---- stages (interface of sharded.CudaStages; CPU tensors)
    def sample(self, n_total, k_evict):
        self.round += 1
        self.keys = [self._keys(b) for b in range(self.B)]
        self.flag = [np.zeros(len(k), bool) for k in self.keys]
        self.resolved = np.zeros(self.B, np.int32)
        p = min(1.0, SAMPLE_MEAN / n_total)
        out = np.zeros((self.B, SAMPLE_CAP), np.uint64)
        counts = np.zeros(self.B, np.int32)
        r = np.random.default_rng(1000 * self.round + self.rank)
        for b in range(self.B):
            take = self.keys[b][r.random(len(self.keys[b])) < p] if p < 1.0 else self.keys[b]
            take = take[:SAMPLE_CAP]
            out[b, :len(take)] = take
            counts[b] = len(take)
        return torch.from_numpy(out.view(np.int64)), torch.from_numpy(counts)

    def bracket(self, gkeys, gcounts, n_total, k_evict):
        gk, gc = gkeys.numpy().view(np.uint64), gcounts.numpy()
        self.lo, self.hi = np.zeros(self.B, np.uint64), np.full(self.B, ALL1)
        for b in range(self.B):
            smp = np.concatenate([gk[w, b, :gc[w, b]] for w in range(gk.shape[0])])
            raw, smp = len(smp), np.sort(smp[:SAMPLE_CAP])
            ns = len(smp)
            if self.distrust:
                self.lo[b] = self.hi[b] = ALL1
                continue
            if ns == 0:
                continue
            if raw == n_total:
                r_lo = r_hi = k_evict
            else:
                mu = k_evict * ns / n_total
                dev = 7.0 * np.sqrt(mu) + 8.0
                r_lo, r_hi = int(np.floor(mu - dev)), int(np.ceil(mu + dev)) + 1
            if r_lo >= 1:
                self.lo[b] = smp[min(r_lo, ns) - 1]
            if r_hi <= ns:
                self.hi[b] = smp[max(r_hi, 1) - 1]

    def filter(self):
        n_below = np.zeros(self.B, np.int64)
        cc = np.zeros(self.B, np.int32)
        self.cand = []
        for b in range(self.B):
            k = self.keys[b]
            below = k < self.lo[b]
            self.flag[b] = below.copy()
            n_below[b] = int(below.sum())
            idx = np.nonzero((k >= self.lo[b]) & (k <= self.hi[b]))[0]
            self.cand.append(idx)
            cc[b] = len(idx)
        return torch.from_numpy(n_below), torch.from_numpy(cc)

    def candidates(self, cap):
        out = np.zeros((self.B, cap, 2), np.int64)
        for b in range(self.B):
            idx = self.cand[b][:cap]
            out[b, :len(idx), 0] = self.keys[b][idx].view(np.int64)
            out[b, :len(idx), 1] = idx
        return torch.from_numpy(out)

    def resolve(self, gcand, gcounts, n_below_global, k_evict, cap, rank):
        gcn, gc, nb = gcand.numpy(), gcounts.numpy(), n_below_global.numpy()
        for b in range(self.B):
            if (gc[:, b] < 0).any():
                continue
            keys = np.concatenate([gcn[w, b, :gc[w, b], 0].view(np.uint64) for w in range(gcn.shape[0])])
            r = int(k_evict - nb[b])
            if r < 0 or r > len(keys):
                continue
            if r > 0:
                tau = np.sort(keys)[r - 1]
                own = self.cand[b]
                self.flag[b][own[self.keys[b][own] <= tau]] = True
            self.resolved[b] = 1
        return torch.from_numpy(self.resolved.copy())

    def new_prefix_rank(self, k_evict):
        return torch.zeros(self.B, dtype=torch.int64), torch.full((self.B,), k_evict, dtype=torch.int64)

    def hist(self, prefix, top):
        out = np.zeros((self.B, 2048), np.int32)
        dbits = min(11, top)
        sh = top - dbits
        pf = prefix.numpy().view(np.uint64)
        for b in range(self.B):
            if self.resolved[b]:
                continue
            k = self.keys[b]
            m = np.ones(len(k), bool) if top >= 64 else (k >> U64(top)) == pf[b]
            d = ((k[m] >> U64(sh)) & U64((1 << dbits) - 1)).astype(np.int64)
            out[b] = np.bincount(d, minlength=2048)[:2048]
        return torch.from_numpy(out)

    def digit(self, hist, prefix, rank, top):
        dbits = min(11, top)
        h, pf, rk = hist.numpy(), prefix.numpy().view(np.uint64), rank.numpy()
        for b in range(self.B):
            cum = np.cumsum(h[b].astype(np.int64))
            if cum[-1] == 0:
                continue
            d = int(np.searchsorted(cum, rk[b], side="left"))
            rk[b] -= (cum[d - 1] if d > 0 else 0)
            pf[b] = (U64(0) if top >= 64 else (pf[b] << U64(dbits))) | U64(d)

    def mark(self, tau):
        t = tau.numpy().view(np.uint64)
        for b in range(self.B):
            if not self.resolved[b]:
                self.flag[b] = self.keys[b] <= t[b]
                self.resolved[b] = 1

    def compact(self):
        out = []
        for b in range(self.B):
            keep = ~self.flag[b]
            for name in ("pos", "lam", "c", "pool"):
                getattr(self, name)[b] = getattr(self, name)[b][keep]
            out.append(int(keep.sum()))
        return out


class ThreadComm:
    """all_gather / all_reduce among `world` threads of one process (emulated ranks).  No device-side waiting: every
    rank's kernels of a stage have been enqueued when the threads meet at the barrier, and tensors are combined with
    ordinary stream-ordered torch operations."""

    class _Shared:
        def __init__(self, world):
            self.world, self.slots, self.barrier = world, [None] * world, threading.Barrier(world)

    def __init__(self, shared, rank):
        self.sh, self.rank, self.world = shared, rank, shared.world

    def all_gather(self, t):
        self.sh.slots[self.rank] = t
        self.sh.barrier.wait()
        out = torch.stack(list(self.sh.slots))
        self.sh.barrier.wait()
        return out

    def all_reduce_sum(self, t):
        g = self.all_gather(t.clone())
        t.copy_(g.sum(0).to(t.dtype))
        return t


def run_ranks_in_threads(world, fn):
    """Runs fn(rank, comm) on `world` threads; re-raises the first exception."""
    shared = ThreadComm._Shared(world)
    errs = [None] * world

    def body(r):
        try:
            fn(r, ThreadComm(shared, r))
        except BaseException as e:          # noqa: BLE001
            errs[r] = e
            shared.barrier.abort()

    ths = [threading.Thread(target=body, args=(r,)) for r in range(world)]
    for t in ths:
        t.start()
    for t in ths:
        t.join()
    for e in errs:
        if e is not None and not isinstance(e, threading.BrokenBarrierError):
            raise e
    for e in errs:
        if e is not None:
            raise e
