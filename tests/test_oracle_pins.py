"""Pins of the CPU oracle against what the paper and the mathematics fix (CPU only).

Each test names the passage it pins.  A plausible mistake in the oracle (dropped term,
wrong sign/index, transposed operand, flipped tie-break) must fail at least one of these.
"""
import functools
import math
import os

import numpy as np
import pytest
import torch

from oracle import trimkv_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


# ----------------------------------------------------------------- score: Eq. (global_score)
def _rows():
    rows = []
    with open(os.path.join(GOLDEN, "score_closed_form.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            b, h, t, i, g = line.split()
            rows.append((float(b), int(h), int(t), int(i), float(g)))
    return rows


@pytest.mark.parametrize("beta,h,t,i,G", _rows())
def test_score_matches_hand_worked_values(beta, h, t, i, G):
    """Hand-worked values of Eq. (global_score) and its limits (tests/golden)."""
    lam32 = np.array([math.log(beta)], np.float32)
    c32 = orc.horizon_term_from_lambda32(lam32, h)
    S = orc.score(lam32, c32, np.array([i]), t)
    assert math.isclose(math.exp(float(S[0])), G, rel_tol=2e-6)


def test_score_equals_direct_sum():
    """exp(S) == sum_{s=t+1}^{t+h} beta^(s-i), Eq. (global_score): pins the age t+1-i and the horizon factor."""
    for h in (1, 2, 3, 5, 8):
        beta = rng.uniform(0.5, 0.99999, size=200)
        t = 300
        pos = rng.integers(1, t + 1, size=200)
        lam32 = np.log(beta).astype(np.float32)
        c32 = orc.horizon_term_from_lambda32(lam32, h)
        S = orc.score(lam32, c32, pos, t).astype(np.float64)
        b = np.exp(lam32.astype(np.float64))
        direct = np.zeros(200)
        for s in range(t + 1, t + h + 1):
            direct += b ** (s - pos)
        np.testing.assert_allclose(np.exp(S), direct, rtol=5e-5)   # fp32 score, ages up to 300
        # the newest token (i = t) has age exactly 1
    lam32 = np.array([-0.25], np.float32)
    S = orc.score(lam32, np.zeros(1, np.float32), np.array([10]), 10)
    assert S[0] == np.float32(-0.25)


def test_score_limits():
    """T-t = 1 gives beta^(t+1-i); T-t -> inf gives beta^(t+1-i)/(1-beta) (text below Eq. (global_score))."""
    beta = rng.uniform(0.1, 0.999, size=100)
    lam = np.log(beta)
    np.testing.assert_allclose(orc.horizon_term(lam, 1), 0.0, atol=0)
    np.testing.assert_allclose(np.exp(orc.horizon_term(lam, 0)), 1.0 / (1.0 - beta), rtol=1e-12)
    # closed form (1-beta^h)/(1-beta) for beta<1
    for h in (2, 4, 7):
        np.testing.assert_allclose(np.exp(orc.horizon_term(lam, h)), (1 - beta ** h) / (1 - beta), rtol=1e-12)
    # beta = 1: the sum has h unit terms; infinite horizon diverges
    assert orc.horizon_term(np.array([0.0]), 4)[0] == math.log(4)
    assert np.isposinf(orc.horizon_term(np.array([0.0]), 0)[0])
    # beta = 0 (lambda = -inf): only the k = 0 term, beta^0 = 1, survives: c = ln 1 = 0 for every horizon
    for h in (1, 2, 5, 0):
        assert orc.horizon_term(np.array([-np.inf]), h)[0] == 0.0


def test_score_is_two_separately_rounded_fp32_ops():
    """The precision contract: fp32 multiply, then fp32 add, not fused and not fp64."""
    lam = np.float32(-1.5230e-8)
    c = np.float32(0.6931472)
    age = 12345
    S = orc.score(np.array([lam]), np.array([c]), np.array([1]), age)   # t+1-i = age
    prod = np.float32(np.float32(age) * lam)
    assert S[0] == np.float32(c + prod)
    # a case where fusing would differ: find one by search
    found = False
    r = np.random.default_rng(7)
    for _ in range(20000):
        lam = np.float32(-r.uniform(1e-3, 1.0))
        c = np.float32(r.uniform(0.0, 0.7))
        a = int(r.integers(1, 5000))
        unfused = np.float32(c + np.float32(np.float32(a) * lam))
        fused = np.float32(np.float64(c) + np.float64(a) * np.float64(lam))
        if unfused != fused:
            S = orc.score(np.array([lam]), np.array([c]), np.array([1]), a)
            assert S[0] == unfused
            found = True
            break
    assert found


# ----------------------------------------------------------------- gate: Sec. 4.1 / 5.1
def test_log_retention_closed_form():
    """lambda = ln sigmoid(s); at the paper's initial bias s = 18: ln(1/(1+e^-18)) = -1.5229979e-8."""
    from decimal import Decimal, getcontext
    getcontext().prec = 60
    exact = -(Decimal(1) + Decimal(-18).exp()).ln()                        # 50-digit reference
    assert abs(float(exact) - (-1.5229979628736e-08)) < 1e-20
    assert math.isclose(float(orc.log_retention(np.array([18.0]))[0]), float(exact), rel_tol=1e-13)
    s = rng.normal(0, 6, size=1000)
    ref = np.log(1.0 / (1.0 + np.exp(-s)))
    np.testing.assert_allclose(orc.log_retention(s), ref, rtol=1e-7, atol=1e-300)   # the naive form cancels for large s
    assert float(orc.log_retention(np.array([-800.0]))[0]) == -800.0      # no overflow for very negative s
    beta, lam, c = orc.retention_terms(np.array([18.0, 0.0, -3.0]), 2)
    np.testing.assert_allclose(beta, 1 / (1 + np.exp(-np.array([18.0, 0.0, -3.0]))), rtol=1e-6)
    np.testing.assert_allclose(np.exp(c.astype(np.float64)), 1 + beta.astype(np.float64), rtol=1e-6)  # h=2: 1+beta
    assert np.all((beta >= 0) & (beta <= 1))                               # beta in [0, 1] (Sec. 2.2)


def test_gate_matches_library_mlp():
    """Sec. 4.1/5.1: sigmoid(w_g^T (W2_h act(W1 x + b1) + b2_h) + b_g) rebuilt from torch.nn.functional in fp64."""
    R, D, dg, de, H = 5, 24, 16, 8, 3
    x = rng.normal(size=(R, D))
    W1 = rng.normal(size=(dg, D)) * 0.3
    b1 = rng.normal(size=dg) * 0.1
    W2 = rng.normal(size=(H, de, dg)) * 0.3
    b2 = rng.normal(size=(H, de)) * 0.1
    w_g = rng.normal(size=de)
    b_g = 0.7
    s = orc.gate_logit(x, W1, b1, W2, b2, w_g, b_g)
    F = torch.nn.functional
    tx = torch.from_numpy(x)
    u = F.silu(F.linear(tx, torch.from_numpy(W1), torch.from_numpy(b1)))
    for h in range(H):
        e = F.linear(u, torch.from_numpy(W2[h]), torch.from_numpy(b2[h]))
        sh = F.linear(e, torch.from_numpy(w_g)[None, :]).squeeze(-1) + b_g
        np.testing.assert_allclose(s[:, h], sh.numpy(), rtol=1e-12, atol=1e-12)
        beta, lam, c = orc.retention_terms(s[:, h], 2)
        np.testing.assert_allclose(beta, torch.sigmoid(sh).numpy(), rtol=1e-6)
        np.testing.assert_allclose(lam, F.logsigmoid(sh).numpy(), rtol=1e-6)


def test_gate_tied_readout_properties():
    """w_g = 0 => beta = sigmoid(b_g) in every (layer, head); equal Proj parameters in two heads => equal beta
    (the readout (w_g, b_g) is shared, Sec. 4.1)."""
    R, D, dg, de, H = 4, 12, 8, 6, 3
    x = rng.normal(size=(R, D))
    W1 = rng.normal(size=(dg, D)); b1 = rng.normal(size=dg)
    W2 = rng.normal(size=(H, de, dg)); b2 = rng.normal(size=(H, de))
    s = orc.gate_logit(x, W1, b1, W2, b2, np.zeros(de), 18.0)
    np.testing.assert_array_equal(s, np.full((R, H), 18.0))
    W2[2] = W2[0]; b2[2] = b2[0]
    s = orc.gate_logit(x, W1, b1, W2, b2, rng.normal(size=de), 1.0)
    np.testing.assert_array_equal(s[:, 0], s[:, 2])
    assert np.abs(s[:, 0] - s[:, 1]).max() > 1e-3


# ----------------------------------------------------------------- selection: Sec. 4.2
def _brute_force_keep(S, pos, layer, head, budget):
    """Independent statement of the rule by a pairwise comparator and Python's sort."""
    def cmp(a, b):
        if S[a] != S[b]:
            return -1 if S[a] > S[b] else 1
        for key in (pos, layer, head):
            if key[a] != key[b]:
                return -1 if key[a] < key[b] else 1
        return 0
    order = sorted(range(len(S)), key=functools.cmp_to_key(cmp))
    return np.array(sorted(order[: min(budget, len(S))]), dtype=np.int64)


@pytest.mark.parametrize("n,distinct", [(1, 1), (17, 3), (200, 5), (1000, 1000), (4096, 40)])
def test_select_matches_brute_force(n, distinct):
    """Keep the M largest under the total order; heavy ties; budgets 0, 1, N-1, N, >N."""
    r = np.random.default_rng(n * 31 + distinct)
    vals = r.normal(size=distinct).astype(np.float32)
    S = vals[r.integers(0, distinct, size=n)]
    L, H = 3, 4
    layer = r.integers(0, L, size=n)
    head = r.integers(0, H, size=n)
    pos = r.integers(1, max(2, n // 4), size=n)
    # make (pos, layer, head) unique per entry as in a real cache
    seen = set(); p2 = pos.copy()
    for j in range(n):
        while (p2[j], layer[j], head[j]) in seen:
            p2[j] += 1
        seen.add((p2[j], layer[j], head[j]))
    for budget in sorted({0, 1, n // 3, n - 1, n, n + 5}):
        if budget < 0:
            continue
        got = orc.select_keep(S, p2, layer, head, budget)
        want = _brute_force_keep(S, p2, layer, head, budget)
        np.testing.assert_array_equal(got, want)
        assert len(got) == min(budget, n)


def test_select_all_equal_scores_closed_form():
    """All scores equal: the kept set is the `budget` smallest (pos, layer, head) triples."""
    L, H, T = 2, 3, 10
    pos, layer, head = np.meshgrid(np.arange(1, T + 1), np.arange(L), np.arange(H), indexing="ij")
    pos, layer, head = pos.ravel(), layer.ravel(), head.ravel()
    perm = np.random.default_rng(3).permutation(len(pos))
    pos, layer, head = pos[perm], layer[perm], head[perm]
    S = np.full(len(pos), -0.125, np.float32)
    budget = 3 * L * H + 4                          # three full positions + 4 triples of position 4
    keep = orc.select_keep(S, pos, layer, head, budget)
    got = sorted(zip(pos[keep], layer[keep], head[keep]))
    want = sorted((p, l, h) for p in range(1, 5) for l in range(L) for h in range(H))[:budget]
    assert got == want
    assert (3 + 1, 0, 0) in got and (4, 1, 1) not in got   # lower layer / lower head win at the boundary


def test_select_signed_zero_and_infinities():
    S = np.array([0.0, -0.0, np.inf, -np.inf, -1.0], np.float32)
    pos = np.array([5, 4, 9, 1, 2]); z = np.zeros(5, np.int64)
    assert list(orc.select_keep(S, pos, z, z, 1)) == [2]
    assert list(orc.select_keep(S, pos, z, z, 2)) == [1, 2]        # -0 == +0; older position (4) wins
    assert list(orc.select_keep(S, pos, z, z, 4)) == [0, 1, 2, 4]
    with pytest.raises(ValueError):
        orc.select_keep(np.array([np.nan], np.float32), [1], [0], [0], 1)


# ----------------------------------------------------------------- the loop: budget, monotonicity, window
def _run_random_cache(L=2, H=3, budget=50, steps=40, prompt=30, seed=0, lam_fn=None, horizon=2):
    r = np.random.default_rng(seed)
    d = 4
    oc = orc.OracleCache(budget, L, H, H * 2, d, horizon=horizon)
    history = []

    def push(n):
        for l in range(L):
            lam = lam_fn(r, n, H) if lam_fn else -np.abs(r.normal(0, 0.05, size=(n, H))).astype(np.float32)
            oc.append(l, r.normal(size=(n, H, d)), r.normal(size=(n, H, d)), lam=lam)

    push(prompt)
    before = {(l, h): set(oc.kept_positions(l, h)) for l in range(L) for h in range(H)}
    oc.score_and_evict()
    history.append((before, {(l, h): set(oc.kept_positions(l, h)) for l in range(L) for h in range(H)}))
    for _ in range(steps):
        push(1)
        before = {(l, h): set(oc.kept_positions(l, h)) for l in range(L) for h in range(H)}
        n_before = oc.total_entries()
        ev = oc.score_and_evict()
        after = {(l, h): set(oc.kept_positions(l, h)) for l in range(L) for h in range(H)}
        assert oc.total_entries() == min(budget, n_before)          # budget invariant, Eq. (2) constraint
        assert ev == max(0, n_before - budget)
        for key in after:
            assert after[key] <= before[key]                         # evicted entries never return, Eq. (1)
        history.append((before, after))
    return oc, history


def test_budget_invariant_and_monotone_eviction():
    _run_random_cache(seed=1)
    _run_random_cache(seed=2, budget=7, prompt=3)      # under budget at first: nothing evicted
    _run_random_cache(seed=3, budget=6 * 3, horizon=0)


def test_equal_retention_reduces_to_sliding_window():
    """All beta equal and < 1, budget = m*L*H: every pool keeps exactly its last m positions."""
    L, H, m = 2, 3, 5
    lam_fn = lambda r, n, H: np.full((n, H), -0.01, np.float32)
    oc, _ = _run_random_cache(L=L, H=H, budget=m * L * H, steps=25, prompt=40, lam_fn=lam_fn)
    t = oc.tokens[0]
    for l in range(L):
        for h in range(H):
            assert list(oc.kept_positions(l, h)) == list(range(t - m + 1, t + 1))


def test_layers_must_agree_on_token_count():
    oc = orc.OracleCache(4, 2, 1, 1, 2)
    oc.append(0, np.zeros((1, 1, 2)), np.zeros((1, 1, 2)), lam=np.zeros((1, 1), np.float32))
    with pytest.raises(RuntimeError):
        oc.score_and_evict()


def test_high_retention_entry_outlives_recent_ones():
    """A longer horizon favours large beta (Sec. 4.2): an old, slowly decaying entry survives newer fast-decaying ones."""
    oc = orc.OracleCache(2, 1, 1, 1, 2, horizon=2)
    lam = np.log(np.array([[0.999]] + [[0.5]] * 5, np.float32))
    oc.append(0, np.zeros((6, 1, 2)), np.zeros((6, 1, 2)), lam=lam)
    oc.score_and_evict()
    assert list(oc.kept_positions(0, 0)) == [1, 6]


# ----------------------------------------------------------------- attention: Sec. 2.1, Eq. (1), Cor. 3.2
def test_attention_full_budget_equals_library_sdpa():
    """Nothing evicted => textbook softmax attention with the 1/sqrt(d) scale (torch SDPA, fp64)."""
    n, d = 37, 16
    q = rng.normal(size=d); K = rng.normal(size=(n, d)); V = rng.normal(size=(n, d))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None, None, None, :], torch.from_numpy(K)[None, None], torch.from_numpy(V)[None, None])
    np.testing.assert_allclose(orc.attention(q, K, V), ref[0, 0, 0].numpy(), rtol=1e-12, atol=1e-14)


def test_attention_special_cases():
    d = 8
    q = rng.normal(size=d); K = rng.normal(size=(9, d)); V = rng.normal(size=(9, d))
    np.testing.assert_allclose(orc.attention(q, K[:1], V[:1]), V[0], rtol=1e-15)        # single entry: o = v
    w = orc.attention_weights(q, K)
    assert math.isclose(w.sum(), 1.0, rel_tol=1e-14) and (w > 0).all()
    p = rng.permutation(9)
    np.testing.assert_allclose(orc.attention(q, K[p], V[p]), orc.attention(q, K, V), rtol=1e-12)  # a sum over a set
    np.testing.assert_array_equal(orc.attention(q, K[:0], V[:0]), np.zeros(d))
    # large logits do not overflow
    assert np.isfinite(orc.attention(q * 1e3, K, V)).all()


def test_gqa_head_mapping_and_cache_attention():
    """Query head j reads the pool of KV head j // g."""
    L, H, Hq, d = 1, 2, 6, 4
    oc = orc.OracleCache(100, L, H, Hq, d)
    K = rng.normal(size=(7, H, d)); V = rng.normal(size=(7, H, d))
    oc.append(0, K, V, lam=np.zeros((7, H), np.float32))
    q = rng.normal(size=(Hq, d))
    o = oc.decode_attention(0, q)
    for j in range(Hq):
        np.testing.assert_allclose(o[j], orc.attention(q[j], K[:, j // 3], V[:, j // 3]), rtol=1e-13)


def test_corollary_3_2_identity():
    """Cor. 3.2: delta^r = (rho_D/rho_U) delta / ((1-delta) + (rho_D/rho_U) delta) for hard eviction r in {0,1}."""
    n, d = 40, 8
    q = rng.normal(size=d); K = rng.normal(size=(n, d))
    useful = np.zeros(n, bool); useful[rng.choice(n, 6, replace=False)] = True
    keep = rng.random(n) < 0.6
    keep[np.flatnonzero(useful)[0]] = True            # at least one useful token retained
    alpha = orc.attention_weights(q, K)
    delta = 1.0 - alpha[useful].sum()
    z = K @ q / math.sqrt(d)
    ez = np.exp(z - z.max())
    rho_U = (keep[useful] * ez[useful]).sum() / ez[useful].sum()
    rho_D = (keep[~useful] * ez[~useful]).sum() / ez[~useful].sum()
    ratio = rho_D / rho_U
    predicted = ratio * delta / ((1 - delta) + ratio * delta)
    alpha_r = orc.attention_weights(q, K[keep])        # attention over the retained set
    delta_r = 1.0 - alpha_r[useful[keep]].sum()
    assert math.isclose(delta_r, predicted, rel_tol=1e-10, abs_tol=1e-14)


# ----------------------------------------------------------------- retention-gated attention: Sec. 2.2
def test_retention_attention_closed_forms():
    """alpha~_i = beta_i^(t-i) e^{z_i} / sum_j ...: hand-checkable cases.

    * beta = 1 everywhere (lambda = 0) recovers standard attention (stated in Sec. 2.2);
    * q = 0 (all z equal): weights are beta_i^(t-i) normalised, here with dyadic beta so the values are exact rationals;
    * the newest token (i = t) carries weight beta^0 = 1 whatever its beta;
    * a uniform shift of all ages (same beta) cancels in the normalisation.
    """
    d = 8
    K = rng.normal(size=(5, d)); V = rng.normal(size=(5, d)); q = rng.normal(size=d)
    pos = np.array([1, 2, 4, 7, 9]); t = 9
    np.testing.assert_allclose(orc.retention_attention(q, K, V, np.zeros(5, np.float32), pos, t), orc.attention(q, K, V), rtol=1e-13)
    # q = 0, beta = 1/2: weights 2^-(t-i) normalised: ages 8, 7, 5, 2, 0
    lam = np.full(5, math.log(0.5), np.float32)
    w = orc.retention_attention_weights(np.zeros(d), K, lam, pos, t)
    raw = np.array([2.0 ** -8, 2.0 ** -7, 2.0 ** -5, 2.0 ** -2, 1.0])
    np.testing.assert_allclose(w, raw / raw.sum(), rtol=1e-6)           # lambda is stored in fp32
    # two entries, worked by hand: beta_1 = 1/4 at age 1, beta_2 = anything at age 0, z_1 = z_2 + ln 8
    K2 = np.array([[math.log(8.0) * math.sqrt(2.0), 0.0], [0.0, 0.0]]); q2 = np.array([1.0, 0.0])
    w2 = orc.retention_attention_weights(q2, K2, np.array([math.log(0.25), -3.0], np.float32), np.array([4, 5]), 5)
    np.testing.assert_allclose(w2, [2.0 / 3.0, 1.0 / 3.0], rtol=1e-6)   # (1/4 * 8) : 1
    # same beta everywhere: adding a constant to every age changes nothing
    lam3 = np.full(5, -0.3, np.float32)
    a = orc.retention_attention(q, K, V, lam3, pos, t)
    b = orc.retention_attention(q, K, V, lam3, pos, t + 11)
    np.testing.assert_allclose(a, b, rtol=1e-9)
    # smaller beta on an old entry lowers its weight (monotone in beta)
    lo = orc.retention_attention_weights(q, K, np.array([-2.0, 0, 0, 0, 0], np.float32), pos, t)
    hi = orc.retention_attention_weights(q, K, np.array([-0.1, 0, 0, 0, 0], np.float32), pos, t)
    assert lo[0] < hi[0] and abs(lo.sum() - 1) < 1e-12


def test_cache_retention_attention_uses_layer_time_and_gqa():
    c = orc.OracleCache(100, 1, 2, 4, 8)
    k = rng.normal(size=(6, 2, 8)); v = rng.normal(size=(6, 2, 8))
    lam = (-rng.uniform(0.01, 0.5, size=(6, 2))).astype(np.float32)
    c.append(0, k, v, lam=lam)
    q = rng.normal(size=(4, 8))
    out = c.decode_attention(0, q, retention_bias=True)
    for j in range(4):
        h = j // 2
        want = orc.retention_attention(q[j], k[:, h], v[:, h], lam[:, h], np.arange(1, 7), 6)
        np.testing.assert_allclose(out[j], want, rtol=1e-12)
    assert np.abs(out - c.decode_attention(0, q)).max() > 1e-3


def test_per_pool_budget_variant():
    """Fixed per-head budget (the TrimKV arm): each pool keeps its own M best entries, independently of the others.
    Equal retention in a pool => that pool keeps its last M positions; a pool with slowly decaying old entries keeps
    them; brute force per pool; pools never exceed M while the global variant moves capacity between them."""
    L, H, M = 2, 2, 5
    c = orc.OracleCache(10 ** 9, L, H, H, 0, horizon=1, per_pool_budget=M)
    g = orc.OracleCache(M * L * H, L, H, H, 0, horizon=1)
    n = 12
    lam = np.full((n, H), -0.1, np.float32)
    lam[:, 1] = -2.0                                   # head 1 forgets fast
    lam[0:3, 1] = -1e-4                                # ... except its three oldest tokens
    kv = np.zeros((n, H, 0))
    for cache in (c, g):
        for l in range(L):
            cache.append(l, kv, kv, lam=lam)
        cache.score_and_evict()
    for l in range(L):
        assert c.kept_positions(l, 0).tolist() == [8, 9, 10, 11, 12]          # sliding window
        assert c.kept_positions(l, 1).tolist() == [1, 2, 3, 11, 12]           # durable old tokens + the newest
        S = orc.score(lam[:, 1], orc.horizon_term_from_lambda32(lam[:, 1], 1), np.arange(1, n + 1), n)
        want = sorted(np.argsort(-S.astype(np.float64), kind="stable")[:M] + 1)
        assert c.kept_positions(l, 1).tolist() == want
    assert (c.lengths() == M).all()
    assert g.lengths().sum() == M * L * H and (g.lengths() != M).any()        # the global budget reallocates


def test_prefill_attention_is_causal_dense_attention_when_nothing_was_evicted():
    """With a budget that evicts nothing, chunked causal attention over the cache equals textbook causal attention
    (torch SDPA with is_causal) over the whole sequence; the last token of a chunk sees what a decode step would."""
    L, H, Hq, d = 1, 2, 4, 8
    c = orc.OracleCache(10 ** 9, L, H, Hq, d)
    T = 11
    k = rng.normal(size=(T, H, d)); v = rng.normal(size=(T, H, d)); q = rng.normal(size=(T, Hq, d))
    lam = np.zeros((T, H), np.float32)
    outs = []
    for a, b in ((0, 4), (4, 5), (5, 11)):                       # chunks of 4, 1 and 6 tokens
        c.append(0, k[a:b], v[a:b], lam=lam[a:b])
        o = c.prefill_attention(0, q[a:b])
        outs.append(o)
        np.testing.assert_allclose(o[-1], c.decode_attention(0, q[b - 1]), rtol=1e-12)
    got = np.concatenate(outs)                                    # [T, Hq, d]
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]               # [1, Hq, T, d]
    tk = torch.from_numpy(np.repeat(k, Hq // H, axis=1)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.repeat(v, Hq // H, axis=1)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-10, atol=1e-12)
    # after an eviction the evicted positions are gone for later chunks, whatever their position
    c2 = orc.OracleCache(6, 1, 1, 1, d)
    lam2 = np.array([[-3.0], [-1e-4], [-3.0], [-1e-4], [-3.0], [-1e-4], [-3.0], [-1e-4]], np.float32)
    c2.append(0, k[:8, :1], v[:8, :1], lam=lam2)
    c2.score_and_evict()
    kept = set(c2.kept_positions(0, 0).tolist())
    assert len(kept) == 6 and {2, 4, 6, 8} <= kept
    c2.append(0, k[8:10, :1], v[8:10, :1], lam=np.zeros((2, 1), np.float32))
    o = c2.prefill_attention(0, q[8:10, :1])
    idx = sorted(p - 1 for p in kept) + [8]
    np.testing.assert_allclose(o[0, 0], orc.attention(q[8, 0], k[idx, 0], v[idx, 0]), rtol=1e-12)


def test_set_horizon_rescoring_closed_forms():
    """Switching the horizon re-scores stored entries (Eq. (global_score)): with h = 1 the score is the myopic
    (t + 1 - i) ln beta, so with beta < 1 equal everywhere the M most recent (position, layer, head) triples survive;
    for two betas, exp(S) must equal the direct sum over s = t+1 .. t+h of beta^(s - i) for the new h; and a cache
    switched to h behaves exactly like one built with h from the start."""
    L, H, d = 2, 2, 4
    rng = np.random.default_rng(5)
    lam = -np.abs(rng.normal(0, 0.3, size=(12, H))).astype(np.float32)
    k = rng.normal(size=(12, H, d)).astype(np.float32)
    a = orc.OracleCache(20, L, H, H, d, horizon=2)
    ref = {h: orc.OracleCache(20, L, H, H, d, horizon=h) for h in (1, 5, 0)}
    for l in range(L):
        a.append(l, k, k, lam=lam)
        for h in ref:
            ref[h].append(l, k, k, lam=lam)
    for h in (1, 5, 0):
        a.set_horizon(h)
        for l in range(L):
            for hh in range(H):
                np.testing.assert_array_equal(a.c[l][hh], ref[h].c[l][hh])
        # direct sum of the definition, fp64
        t = 12
        i = a.pos[0][0].astype(np.float64)
        beta = np.exp(a.lam[0][0].astype(np.float64))
        S = orc.score(a.lam[0][0], a.c[0][0], a.pos[0][0], t).astype(np.float64)
        if h > 0:
            direct = sum(beta ** (s - i) for s in range(t + 1, t + h + 1))
        else:
            direct = beta ** (t + 1 - i) / (1.0 - beta)
        np.testing.assert_allclose(np.exp(S), direct, rtol=2e-6)
    a.set_horizon(1)
    assert all((a.c[l][hh] == 0).all() for l in range(L) for hh in range(H))
    a.score_and_evict()
    ref[1].score_and_evict()
    for l in range(L):
        for hh in range(H):
            np.testing.assert_array_equal(a.kept_positions(l, hh), ref[1].kept_positions(l, hh))
    # equal beta < 1 and h = 1: pure recency, 20 = 5 * L * H entries -> the last 5 positions of every pool
    b = orc.OracleCache(20, L, H, H, d, horizon=3)
    for l in range(L):
        b.append(l, k, k, lam=np.full((12, H), -0.1, np.float32))
    b.set_horizon(1)
    b.score_and_evict()
    for l in range(L):
        for hh in range(H):
            np.testing.assert_array_equal(b.kept_positions(l, hh), np.arange(8, 13))


def test_rounding_contract_case_discriminates_fused_and_fp64_scores():
    """The inputs of the GPU score-rounding test: in EVERY sequence the kept set under the contract's score (fp32
    multiply, then fp32 add) differs from the kept set under a fused multiply-add and under fp64 evaluation, so a kernel
    that contracts the two operations, or scores in higher precision, cannot reproduce the oracle's sets."""
    import util_parity as up
    lam, c, budget = up.rounding_contract_case(seed=5, B=24, n=48, L=2, H=2)
    want = up.rounding_contract_kept_sets(lam, c, budget, "contract")
    fused = up.rounding_contract_kept_sets(lam, c, budget, "fused")
    fp64 = up.rounding_contract_kept_sets(lam, c, budget, "fp64")
    for b in range(lam.shape[1]):
        assert len(want[b]) == budget
        assert want[b] != fused[b] and want[b] != fp64[b]
        assert len(want[b] ^ fused[b]) == 2 and len(want[b] ^ fp64[b]) == 2      # exactly the pair's two members swap
