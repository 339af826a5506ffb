"""Plain CPU oracle of the global retention-based KV eviction decode loop.

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of
what the hot path computes, written from the paper's definitions with numpy.  It
shares no code with the CUDA library and is never imported by it.  Floating point
is fp64 except where a precision is part of the method's contract (the fp32
retention terms stored with an entry and the fp32 score, see `score`).

What each function follows:

* `gate_logit`, `retention_terms`  -- Sec. 4.1 "Weight-tied retention gates"
  (beta = sigmoid(w_g^T Proj_{l,h}(x) + b_g)) and Sec. 5.1 "Implementation details"
  (Proj is a two-layer MLP of hidden width d_g; (w_g, b_g) tied over layers/heads).
* `horizon_term`, `score`          -- Eq. (global_score), Sec. 4.2, in log space.
* `select_keep`                    -- Sec. 4.2 eviction rule: keep the M_global
  largest scores over all layers and heads (full sort = the plain definition).
* `attention`, `attention_weights` -- Sec. 2.1 softmax attention restricted to the
  retained set (Eq. (1) with r in {0,1}).
* `retention_attention`, `retention_attention_weights` -- Sec. 2.2 retention-gated attention
  (weights beta_i^(t-i) e^{z_i}), an option of the decode attention.
* `OracleCache`                    -- the per-step loop: append, score, evict, attend.

Parity pins: every function here is pinned by tests/test_oracle_pins.py except the
items the paper leaves open, which are readings and are marked "parity unpinned":
  - the gate's internals (activation = SiLU, first layer shared by a layer's heads,
    head-specific second layer of width d_e, biases),
  - whether the newest token competes in the ranking (it does here),
  - the direction of the tie-break (older position, lower layer, lower head win).
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
F64 = np.float64


# --------------------------------------------------------------------------- gate
def _silu(z):
    return z / (1.0 + np.exp(-z))


def gate_logit(x, W1, b1, W2, b2, w_g, b_g):
    """Pre-sigmoid gate score s[r, h] = w_g . Proj_{l,h}(x_r) + b_g  (Sec. 4.1).

    Proj_{l,h}(x) = W2[h] @ act(W1 @ x + b1) + b2[h]  (two-layer MLP, Sec. 5.1).
    x [R, D]; W1 [d_g, D]; b1 [d_g]; W2 [H, d_e, d_g]; b2 [H, d_e]; w_g [d_e].
    All arithmetic in fp64.
    """
    x = np.asarray(x, F64)
    u = _silu(x @ np.asarray(W1, F64).T + np.asarray(b1, F64))            # [R, d_g]
    e = np.einsum("rj,hkj->rhk", u, np.asarray(W2, F64)) + np.asarray(b2, F64)  # [R, H, d_e]
    return e @ np.asarray(w_g, F64) + F64(b_g)                            # [R, H]


def log_retention(s):
    """lambda = ln(beta) = ln(sigmoid(s)) = -softplus(-s), fp64, stable for any s."""
    s = np.asarray(s, F64)
    return -(np.log1p(np.exp(-np.abs(s))) + np.maximum(-s, 0.0))


def horizon_term(lam, horizon):
    """c = ln( sum_{k=0}^{h-1} beta^k ) with beta = exp(lam); h = `horizon` = T - t.

    This is the beta-only factor of Eq. (global_score): the closed form
    (1 - beta^h) / (1 - beta) for beta < 1, written as the finite sum so that it is
    also defined at beta = 1 (where it equals h).  horizon == 0 means T - t -> inf:
    c = -ln(1 - beta) (the limit stated below the equation); +inf at beta = 1.
    """
    lam = np.asarray(lam, F64)
    if horizon == 0:
        with np.errstate(divide="ignore"):
            return -np.log(-np.expm1(lam))
    acc = np.ones_like(lam)                      # k = 0: beta^0 = 1 for every beta, beta = 0 (lam = -inf) included
    for k in range(1, int(horizon)):
        acc = acc + np.exp(k * lam)
    return np.log(acc)


def retention_terms(s, horizon):
    """(beta, lambda, c) of a gate logit s, each rounded once to fp32 (what an entry stores)."""
    s = np.asarray(s, F64)
    beta = np.where(s >= 0, 1.0 / (1.0 + np.exp(-np.abs(s))), np.exp(-np.abs(s)) / (1.0 + np.exp(-np.abs(s))))
    lam = log_retention(s)
    c = horizon_term(lam, horizon)
    return beta.astype(F32), lam.astype(F32), c.astype(F32)


def horizon_term_from_lambda32(lam32, horizon):
    """c for a caller-supplied fp32 lambda: fp64 evaluation of `horizon_term`, rounded to fp32."""
    return horizon_term(np.asarray(lam32, F32).astype(F64), horizon).astype(F32)


# -------------------------------------------------------------------------- score
def score(lam32, c32, pos, t):
    """Log-space retention score S = ln G~_{l,h,i}(t) of Eq. (global_score).

    G~ = beta^(t+1-i) * sum_{k<h} beta^k  =>  S = (t+1-i) * lambda + c.
    `pos` is the 1-based token position i, `t` the number of tokens seen so far.
    Precision contract: the age is exact in fp32, then ONE fp32 multiply and ONE fp32
    add, each rounded to nearest even, never fused.  Inputs are the fp32 (lambda, c)
    stored with the entry.
    """
    lam32 = np.asarray(lam32, F32)
    c32 = np.asarray(c32, F32)
    age = (np.int64(t) + 1 - np.asarray(pos, np.int64)).astype(F32)
    prod = (age * lam32).astype(F32)
    return (c32 + prod).astype(F32)


# ------------------------------------------------------------------------- select
def select_keep(S, pos, layer, head, budget):
    """Indices (into the given arrays) of the min(budget, N) entries that are kept.

    Sec. 4.2: keep the M_global largest scores across all layers and heads.  Ties are
    resolved by a total order: higher score first; equal scores -> smaller position
    first; then smaller layer; then smaller head.  The kept entries are the first
    `budget` of the fully sorted list.
    """
    S = np.asarray(S, F32)
    if np.isnan(S).any():
        raise ValueError("NaN score")
    n = S.shape[0]
    keep_n = int(min(int(budget), n))
    # np.lexsort: LAST key is the primary one.  -S ascending == S descending.
    order = np.lexsort((np.asarray(head), np.asarray(layer), np.asarray(pos), -S.astype(F64)))
    return np.sort(order[:keep_n])


# ---------------------------------------------------------------------- attention
def attention_weights(q, K):
    """alpha_i = softmax_i(q . k_i / sqrt(d)) over the rows of K  (Sec. 2.1), fp64."""
    q = np.asarray(q, F64)
    K = np.asarray(K, F64)
    z = (K @ q) / np.sqrt(F64(q.shape[-1]))
    z = z - z.max()
    w = np.exp(z)
    return w / w.sum()


def attention(q, K, V):
    """o = sum_i alpha_i v_i over the retained entries (Eq. (1), r in {0,1}), fp64.

    An empty retained set yields zeros (the definition's empty sum).
    """
    V = np.asarray(V, F64)
    if V.shape[0] == 0:
        return np.zeros(V.shape[-1], F64)
    return attention_weights(q, K) @ V


def retention_attention_weights(q, K, lam32, pos, t):
    """alpha~_i = beta_i^(t-i) e^{z_i} / sum_j beta_j^(t-j) e^{z_j}  (Sec. 2.2, retention-gated attention), fp64.

    z_i = q . k_i / sqrt(d); beta_i^(t-i) = exp((t - i) * lambda_i) with the entry's stored fp32 lambda_i = ln beta_i and
    its 1-based position i; t = number of tokens seen.  The newest token (i = t) has weight beta^0 = 1; lambda = 0
    everywhere gives back plain softmax attention.
    """
    q = np.asarray(q, F64)
    K = np.asarray(K, F64)
    z = (K @ q) / np.sqrt(F64(q.shape[-1]))
    z = z + (F64(t) - np.asarray(pos, F64)) * np.asarray(lam32, F32).astype(F64)
    z = z - z.max()
    w = np.exp(z)
    return w / w.sum()


def retention_attention(q, K, V, lam32, pos, t):
    """o~ = sum_i alpha~_i v_i over the retained entries (Sec. 2.2); zeros for an empty set."""
    V = np.asarray(V, F64)
    if V.shape[0] == 0:
        return np.zeros(V.shape[-1], F64)
    return retention_attention_weights(q, K, lam32, pos, t) @ V


# ------------------------------------------------------------------ the step loop
class OracleCache:
    """One sequence's budgeted cache: per-(layer, head) sets of entries, ordered by position.

    Follows the per-step loop: a token's retention is estimated once when it enters
    the cache (Sec. 3.2), every entry is re-scored at eviction time t and the
    M_global best over all (layer, head) pools survive (Sec. 4.2); evicted entries
    never return (monotone r, Eq. (1)).
    """

    def __init__(self, budget, layers, kv_heads, q_heads, head_dim, horizon=2, per_pool_budget=0):
        self.budget = int(budget)
        # > 0: the fixed-budget variant the paper compares with (TrimKV, Sec. 2.2 / 5.2: a budget of M entries for
        # each attention head instead of one global budget): every pool keeps its own M best entries
        self.per_pool_budget = int(per_pool_budget)
        self.L, self.H, self.Hq, self.d = int(layers), int(kv_heads), int(q_heads), int(head_dim)
        assert self.Hq % self.H == 0
        self.g = self.Hq // self.H
        self.horizon = int(horizon)
        self.tokens = [0] * self.L                      # tokens appended per layer
        # per pool: parallel arrays
        self.pos = [[np.zeros(0, np.int64) for _ in range(self.H)] for _ in range(self.L)]
        self.lam = [[np.zeros(0, F32) for _ in range(self.H)] for _ in range(self.L)]
        self.c = [[np.zeros(0, F32) for _ in range(self.H)] for _ in range(self.L)]
        self.K = [[np.zeros((0, self.d), F64) for _ in range(self.H)] for _ in range(self.L)]
        self.V = [[np.zeros((0, self.d), F64) for _ in range(self.H)] for _ in range(self.L)]
        self.gate = None

    # gate parameters: per layer (W1, b1, W2, b2); shared (w_g, b_g)
    def set_gate(self, layer_params, w_g, b_g):
        self.gate = (layer_params, np.asarray(w_g, F64), float(b_g))

    def gate_outputs(self, layer, x):
        """(beta, lambda, c) fp32 arrays [n, H] for the rows of x [n, D]."""
        params, w_g, b_g = self.gate
        W1, b1, W2, b2 = params[layer]
        s = gate_logit(x, W1, b1, W2, b2, w_g, b_g)
        return retention_terms(s, self.horizon)

    def append(self, layer, k, v, x=None, lam=None, c=None):
        """Append n tokens to every pool of `layer`.  k, v: [n, H, d].

        Retention comes from the gate on x [n, D], or is supplied as fp32 lam [n, H]
        (and optionally c [n, H]; otherwise c is derived from lam).
        Token j of the call gets the 1-based position tokens[layer] + j + 1.
        """
        k = np.asarray(k)
        v = np.asarray(v)
        n = k.shape[0]
        if x is not None:
            _, lam, c = self.gate_outputs(layer, x)
        else:
            lam = np.asarray(lam, F32)
            c = horizon_term_from_lambda32(lam, self.horizon) if c is None else np.asarray(c, F32)
        if np.isnan(lam).any() or np.isnan(c).any():
            raise ValueError("non-finite retention")
        base = self.tokens[layer]
        newpos = base + 1 + np.arange(n, dtype=np.int64)
        for h in range(self.H):
            self.pos[layer][h] = np.concatenate([self.pos[layer][h], newpos])
            self.lam[layer][h] = np.concatenate([self.lam[layer][h], lam[:, h]])
            self.c[layer][h] = np.concatenate([self.c[layer][h], c[:, h]])
            self.K[layer][h] = np.concatenate([self.K[layer][h], k[:, h, :].astype(F64)])
            self.V[layer][h] = np.concatenate([self.V[layer][h], v[:, h, :].astype(F64)])
        self.tokens[layer] = base + n

    def set_horizon(self, horizon):
        """Switch the horizon h = T - t of Eq. (global_score) for stored and future entries: the beta-only term
        c = ln sum_{k<h} beta^k of every entry is recomputed from its stored fp32 lambda (h = 1: c = 0, the myopic
        score; h = 0: the h -> inf limit -ln(1 - beta))."""
        self.horizon = int(horizon)
        for l in range(self.L):
            for h in range(self.H):
                self.c[l][h] = horizon_term_from_lambda32(self.lam[l][h], self.horizon)

    def total_entries(self):
        return sum(len(self.pos[l][h]) for l in range(self.L) for h in range(self.H))

    def flat(self):
        """All entries as flat arrays (S needs t): returns (lam, c, pos, layer, head)."""
        lam = np.concatenate([self.lam[l][h] for l in range(self.L) for h in range(self.H)])
        c = np.concatenate([self.c[l][h] for l in range(self.L) for h in range(self.H)])
        pos = np.concatenate([self.pos[l][h] for l in range(self.L) for h in range(self.H)])
        layer = np.concatenate([np.full(len(self.pos[l][h]), l, np.int64) for l in range(self.L) for h in range(self.H)])
        head = np.concatenate([np.full(len(self.pos[l][h]), h, np.int64) for l in range(self.L) for h in range(self.H)])
        return lam, c, pos, layer, head

    def score_and_evict(self):
        """One eviction round at time t = tokens appended so far (same in every layer)."""
        t = self.tokens[0]
        if any(tt != t for tt in self.tokens):
            raise RuntimeError("layers hold different token counts")
        if self.per_pool_budget > 0:
            evicted = 0
            for l in range(self.L):
                for h in range(self.H):
                    m = len(self.pos[l][h])
                    if m <= self.per_pool_budget:
                        continue
                    S = score(self.lam[l][h], self.c[l][h], self.pos[l][h], t)
                    z = np.zeros(m, np.int64)
                    keep = select_keep(S, self.pos[l][h], z, z, self.per_pool_budget)
                    for name in ("pos", "lam", "c", "K", "V"):
                        arr = getattr(self, name)
                        arr[l][h] = arr[l][h][keep]
                    evicted += m - self.per_pool_budget
            return evicted
        n = self.total_entries()
        if n <= self.budget:
            return 0
        lam, c, pos, layer, head = self.flat()
        S = score(lam, c, pos, t)
        keep = select_keep(S, pos, layer, head, self.budget)
        mask = np.zeros(n, bool)
        mask[keep] = True
        off = 0
        for l in range(self.L):
            for h in range(self.H):
                m = len(self.pos[l][h])
                sel = mask[off:off + m]
                self.pos[l][h] = self.pos[l][h][sel]
                self.lam[l][h] = self.lam[l][h][sel]
                self.c[l][h] = self.c[l][h][sel]
                self.K[l][h] = self.K[l][h][sel]
                self.V[l][h] = self.V[l][h][sel]
                off += m
        return n - self.budget

    def prefill_attention(self, layer, q):
        """Causal attention of the chunk just appended to `layer` (its last n tokens), q [n, Hq, d] -> [n, Hq, d] fp64.

        Token j of the chunk sits at position p = tokens[layer] - n + j + 1 and attends to the retained entries with
        position <= p (Sec. 2.1: C_t = {1..t}, restricted to the retained set as in Eq. (1)): everything kept from before
        the chunk plus the chunk's own tokens up to itself.
        """
        q = np.asarray(q, F64)
        n = q.shape[0]
        base = self.tokens[layer] - n
        out = np.zeros((n, self.Hq, self.d), F64)
        for j in range(n):
            p = base + j + 1
            for hq in range(self.Hq):
                h = hq // self.g
                vis = self.pos[layer][h] <= p
                out[j, hq] = attention(q[j, hq], self.K[layer][h][vis], self.V[layer][h][vis])
        return out

    def lengths(self):
        return np.array([[len(self.pos[l][h]) for h in range(self.H)] for l in range(self.L)], np.int32)

    def kept_positions(self, layer, head):
        return self.pos[layer][head].copy()

    def decode_attention(self, layer, q, retention_bias=False):
        """q [Hq, d] -> o [Hq, d] fp64; query head j reads the pool of KV head j // g.

        retention_bias: use the retention-gated weights of Sec. 2.2 (beta_i^(t-i) e^{z_i}) instead of the plain softmax
        over the retained set (Eq. (1)); t = tokens appended to this layer so far.
        """
        q = np.asarray(q, F64)
        out = np.zeros((self.Hq, self.d), F64)
        for j in range(self.Hq):
            h = j // self.g
            if retention_bias:
                out[j] = retention_attention(q[j], self.K[layer][h], self.V[layer][h], self.lam[layer][h],
                                             self.pos[layer][h], self.tokens[layer])
            else:
                out[j] = attention(q[j], self.K[layer][h], self.V[layer][h])
        return out
