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
        self.gpu.check_invariants()               # block tables, page records, free stacks, positions: all consistent

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


# ------------------------------------------------------------------------------------------- score rounding contract
def _score_variants(lam, c, age):
    """(unfused fp32 multiply then add, fused = one rounding of the exact value, exact in fp64) for fp32 lam, c."""
    lam, c = np.float32(lam), np.float32(c)
    unfused = np.float32(c + np.float32(np.float32(age) * lam))
    exact = np.float64(c) + np.float64(age) * np.float64(lam)      # the product is exact in fp64 (24 + 6 bits)
    return unfused, np.float32(exact), exact


def rounding_sensitive_pair(r, age1, age2, want_tie=False):
    """Two entries (lam1, c1), (lam2, c2) of ages age1, age2 whose ORDER under the contract's score (fp32 multiply, then
    fp32 add, each rounded) differs from their order under a fused multiply-add and under fp64 evaluation.
    want_tie: the contract's scores tie exactly while the other two evaluations rank the pair strictly.
    Returns (lam1, c1, lam2, c2, sign): sign = +1 if entry 1 outranks entry 2 under the contract, -1 if entry 2 does;
    for a tie, sign is the order under the OTHER two evaluations (+1: they rank entry 1 first)."""
    for _ in range(200000):
        lam1 = np.float32(-r.uniform(1e-3, 0.1))
        lam2 = np.float32(-r.uniform(1e-3, 0.1))
        c1 = np.float32(r.uniform(0.0, 0.7))
        s1, f1, e1 = _score_variants(lam1, c1, age1)
        c2 = np.float32(np.float64(s1) - np.float64(age2) * np.float64(lam2))
        for _step in range(int(r.integers(0, 4))):
            c2 = np.nextafter(c2, np.float32(r.choice([-1.0, 1.0]) * 10), dtype=np.float32)
        s2, f2, e2 = _score_variants(lam2, c2, age2)
        su, sf, se = np.sign(np.float64(s1) - np.float64(s2)), np.sign(np.float64(f1) - np.float64(f2)), np.sign(e1 - e2)
        if want_tie:
            if su == 0 and sf != 0 and sf == se:
                return lam1, c1, lam2, c2, int(sf)
        elif su != 0 and sf == -su and se == -su:
            return lam1, c1, lam2, c2, int(su)
    raise AssertionError("no rounding-sensitive pair found")


def rounding_contract_case(seed, B, n, L, H):
    """Per sequence: n tokens in each of L x H pools.  One pair of entries per sequence is rounding-sensitive (see above)
    and scores in (-6, 1); half of the other entries score +8, the rest -8 (lambda = 0, c = +-8).  With a budget of
    (#high + 1) entries the kept set contains the high entries plus the ONE member of the pair that the score's rounding
    contract ranks first.  Returns lam, c [L][B, n, H] fp32 and the budget."""
    r = np.random.default_rng(seed)
    lam = np.zeros((L, B, n, H), np.float32)
    c = np.zeros((L, B, n, H), np.float32)
    total = n * L * H
    n_high = (total - 2) // 2
    t = n                                                       # eviction time: every layer holds n tokens
    nice = [p for p in range(n) if (t - p) >= 3 and ((t - p) & (t - p - 1))]        # 0-based token index; age = t - p
    for b in range(B):
        slots = [(l, p, h) for l in range(L) for p in range(n) for h in range(H)]
        while True:
            i1, i2 = r.choice(len(slots), size=2, replace=False)
            (l1, p1, h1), (l2, p2, h2) = slots[i1], slots[i2]
            if p1 in nice and p2 in nice and p1 != p2:
                break
        want_tie = (b % 5 == 4)
        if want_tie and (p2, l2, h2) < (p1, l1, h1):            # entry 1 = the member the tie-break keeps (older, ...)
            (l1, p1, h1), (l2, p2, h2), i1, i2 = (l2, p2, h2), (l1, p1, h1), i2, i1
        a1, a2 = t - p1, t - p2                                 # age t + 1 - i with i = p + 1
        while True:
            lm1, c1, lm2, c2, sign = rounding_sensitive_pair(r, a1, a2, want_tie)
            if not want_tie or sign < 0:                        # a tie only tells if the other evaluations prefer entry 2
                break
        others = [s for j, s in enumerate(slots) if j not in (i1, i2)]
        order = r.permutation(len(others))
        for rank, j in enumerate(order):
            l, p, h = others[j]
            c[l, b, p, h] = 8.0 if rank < n_high else -8.0
        lam[l1, b, p1, h1], c[l1, b, p1, h1] = lm1, c1
        lam[l2, b, p2, h2], c[l2, b, p2, h2] = lm2, c2
    return lam, c, n_high + 1


def rounding_contract_kept_sets(lam, c, budget, variant):
    """Kept (layer, token, head) triples per sequence of a rounding_contract_case under a score evaluation:
    "contract" = the oracle's score; "fused" / "fp64" = the two evaluations a kernel could slip into."""
    L, B, n, H = lam.shape
    t = n
    lay, tok, hd = [a.reshape(-1) for a in np.meshgrid(np.arange(L), np.arange(n), np.arange(H), indexing="ij")]
    pos = tok + 1
    out = []
    for b in range(B):
        lm, cc = lam[:, b].reshape(-1), c[:, b].reshape(-1)
        if variant == "contract":
            S = orc.score(lm, cc, pos, t)
            keep = orc.select_keep(S, pos, lay, hd, budget)
        else:
            exact = cc.astype(np.float64) + (t + 1 - pos).astype(np.float64) * lm.astype(np.float64)
            S = exact.astype(np.float32).astype(np.float64) if variant == "fused" else exact
            order = np.lexsort((hd, lay, pos, -S))             # the oracle's total order on the variant's scores
            keep = np.sort(order[:budget])
        out.append(set(zip(lay[keep].tolist(), tok[keep].tolist(), hd[keep].tolist())))
    return out
