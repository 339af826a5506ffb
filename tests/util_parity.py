"""Helpers that drive the CUDA library and the CPU oracle with the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import trimkv_oracle as orc
from paper_2605_09649_b200 import binding, workloads


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy()


class Pair:
    """A CUDA cache and one oracle cache per (sampled) sequence, fed identical inputs."""

    def __init__(self, w: workloads.Workload, device="cuda", oracle_seqs=None, oracle_kv=True, **overrides):
        self.w = w
        self.dev = device
        self.retention_bias = bool(overrides.get("retention_bias", False))
        self.gpu = binding.TrimKV.from_workload(w, **overrides)
        self.seqs = list(range(w.batch)) if oracle_seqs is None else list(oracle_seqs)
        self.oracle_kv = oracle_kv
        d = w.head_dim if oracle_kv else 0
        self.orc = {b: orc.OracleCache(w.budget_entries, w.layers, w.kv_heads, w.q_heads, d, horizon=w.horizon,
                                       per_pool_budget=int(overrides.get("per_pool_budget", 0)))
                    for b in self.seqs}

    def close(self):
        self.gpu.close()

    def append(self, layer, k, v, lam_np, c_np):
        """k, v: device tensors [B, n, H, d]; lam_np, c_np: float32 numpy [B, n, H] (the oracle's values)."""
        lam_t = torch.from_numpy(np.ascontiguousarray(lam_np)).to(self.dev)
        c_t = torch.from_numpy(np.ascontiguousarray(c_np)).to(self.dev)
        self.gpu.append(layer, k, v, lam=lam_t, c=c_t)
        for b in self.seqs:
            if self.oracle_kv:
                kk, vv = to_np(k[b]), to_np(v[b])
            else:
                kk = vv = np.zeros((k.shape[1], self.w.kv_heads, 0), np.float32)
            self.orc[b].append(layer, kk, vv, lam=lam_np[b], c=c_np[b])

    def evict(self):
        self.gpu.score_and_evict()
        for b in self.seqs:
            self.orc[b].score_and_evict()

    def check_sets(self):
        """Bit-exact kept sets: lengths and sorted positions of every pool of every sampled sequence."""
        w = self.w
        lens = self.gpu.lengths().numpy()
        for b in self.seqs:
            want = self.orc[b].lengths()
            np.testing.assert_array_equal(lens[b], want, err_msg=f"pool lengths differ in sequence {b}")
            for l in range(w.layers):
                for h in range(w.kv_heads):
                    got = self.gpu.kept(b, l, h, int(want[l, h]) + 1).numpy()
                    np.testing.assert_array_equal(got, self.orc[b].kept_positions(l, h),
                                                  err_msg=f"kept set differs in pool ({b},{l},{h})")
        self.gpu.sync_status()

    def check_attention(self, layer, q, atol):
        """q [B, Hq, d] device tensor; compares the CUDA output with the oracle's fp64 result."""
        out = self.gpu.decode_attention(layer, q)
        got = to_np(out)
        for b in self.seqs:
            want = self.orc[b].decode_attention(layer, to_np(q[b]), retention_bias=self.retention_bias)
            err = np.abs(got[b] - want).max()
            assert err <= atol, f"attention error {err} > {atol} in sequence {b}, layer {layer}"
        return out


def oracle_retention(lam32: np.ndarray, horizon: int):
    return orc.horizon_term_from_lambda32(lam32, horizon)


def random_lambda(shape, seed, distinct=0, scale=0.05):
    """Seeded negative log-retentions; `distinct` > 0 draws from that many values (heavy score ties)."""
    r = np.random.default_rng(seed)
    if distinct > 0:
        vals = -np.abs(r.normal(0, scale, size=distinct)).astype(np.float32)
        return vals[r.integers(0, distinct, size=shape)]
    return -np.abs(r.normal(0, scale, size=shape)).astype(np.float32)
