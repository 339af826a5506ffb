"""Full-size parity: the named workloads at their full shapes, cache at its budget, stepped with
trimkv_decode_step_all exactly as bench.py does (all layers per call, gate on x, two internal streams).

The oracle cannot run a whole step at these sizes in seconds, so one sequence is sampled and checked in full for
the integer work (the kept set of every one of its pools, bit-exact, against the oracle's full sort over the same
fp32 retention terms), sampled pools are checked for attention (the oracle's fp64 attention over the pool's rows
read back from the device), a sampled layer for the gate, and every sequence for the budget invariant.
"""
import numpy as np
import pytest
import torch

from oracle import trimkv_oracle as orc
from paper_2605_09649_b200 import binding, workloads
from util_parity import to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _prefill(cache, w, bank, seed, context):
    done = 0
    while done < context:
        n = min(w.chunk, context - done)
        for l in range(w.layers):
            x = workloads.hidden_states(w, seed, l, done, n, device=DEV)
            _, k, v = workloads.project_qkv(w, bank, l, x)
            cache.append(l, k, v, x=x)
        cache.score_and_evict()
        done += n
    cache.sync_status()


def _step_inputs(w, bank, seed, token):
    xs, ks, vs, qs = [], [], [], []
    for l in range(w.layers):
        x = workloads.hidden_states(w, seed, l, token, 1, device=DEV)
        q, k, v = workloads.project_qkv(w, bank, l, x)
        xs.append(x[:, 0]); ks.append(k[:, 0]); vs.append(v[:, 0]); qs.append(q[:, 0])
    return [torch.stack(t).contiguous() for t in (xs, ks, vs, qs)]


# context: enough tokens to fill the budget (the cache is then in the same state class as after the full prompt,
# and the set-up stays short); the llama shape also runs its full 32K prompt
# skew > 0: per-(layer, head) gate-logit offsets N(0, skew) (through b2, as `bench.py --skew` applies them): retention then
# differs by orders of magnitude between heads, pool lengths run from 0 to tens of thousands of entries, long pools are
# cut into many work items and the attention kernel's in-kernel merge is live
CASES = [("llama8b_32k", 32768, 0, 0.0), ("qwen_vl_16k", 4096, 2, 0.0), ("stress_128k", 9216, 0, 0.0),
         ("multiturn", 2048, 5, 0.0), ("llama8b_32k", 32768, 3, 3.0)]


@pytest.mark.parametrize("name,context,seq,skew", CASES)
def test_full_size_step_matches_oracle_on_samples(name, context, seq, skew):
    w = workloads.WORKLOADS[name]
    seed = 0
    LH = w.layers * w.kv_heads
    cache = binding.TrimKV.from_workload(w)
    per_layer, w_g = workloads.gate_params(w, seed, device=DEV)
    if skew > 0:
        off = workloads.head_logit_offsets(w, seed, skew, device=DEV)
        wn = w_g / (w_g * w_g).sum()
        per_layer = [(W1, b1, W2, (b2 + off[l][:, None] * wn[None, :]).contiguous())
                     for l, (W1, b1, W2, b2) in enumerate(per_layer)]
    for l, p in enumerate(per_layer):
        cache.set_gate(l, *p)
    cache.set_shared_projection(w_g, w.b_g)
    bank = workloads.ProjectionBank(w, seed, device=DEV)
    _prefill(cache, w, bank, seed, context)
    assert int(cache.lengths()[seq].sum()) == min(w.budget_entries, context * LH)
    # two warm steps so that the cache is in its steady decode state, then the checked step
    for i in range(2):
        X, K, V, Q = _step_inputs(w, bank, seed, context + i)
        cache.decode_step_all(K, V, Q, torch.empty_like(Q), x=X)
    t = context + 2                                      # tokens seen before the checked step
    rng = np.random.default_rng(7)
    sample_pools = [(int(rng.integers(w.layers)), int(rng.integers(w.kv_heads))) for _ in range(4)]

    # ---- state of the sampled sequence before the step
    lens = cache.lengths()[seq].numpy()
    if skew > 0:                                         # ragged pools: also the longest and the shortest non-empty pool
        assert lens.max() > 8 * max(int(lens[lens > 0].min()), 1) and lens.max() > 16384
        longest = np.unravel_index(np.argmax(lens), lens.shape)
        shortest = np.unravel_index(np.argmin(np.where(lens > 0, lens, 1 << 30)), lens.shape)
        sample_pools += [(int(longest[0]), int(longest[1])), (int(shortest[0]), int(shortest[1]))]
    cap = int(lens.max()) + 2
    before = {}
    for l in range(w.layers):
        for h in range(w.kv_heads):
            kv = (l, h) in sample_pools
            pos, lam, c, k, v = cache.pool(seq, l, h, cap, with_kv=kv)
            before[(l, h)] = (pos.numpy().astype(np.int64), lam.numpy(), c.numpy(),
                              to_np(k).astype(np.float64) if kv else None, to_np(v).astype(np.float64) if kv else None)

    X, K, V, Q = _step_inputs(w, bank, seed, t)
    out = torch.empty_like(Q)
    cache.decode_step_all(K, V, Q, out, x=X)
    cache.sync_status()

    # ---- gate of a sampled layer against the oracle (fp64), and the terms the new entries received
    lg = int(rng.integers(w.layers))
    W1, b1, W2, b2 = [to_np(p).astype(np.float64) for p in per_layer[lg]]
    s = orc.gate_logit(to_np(X[lg]), W1, b1, W2, b2, to_np(w_g), w.b_g)
    _, olam, oc = orc.retention_terms(s, w.horizon)
    _, glam, gc = cache.gate(lg, X[lg][:, None].contiguous())
    np.testing.assert_allclose(to_np(glam)[:, 0], olam, rtol=1e-5, atol=0)
    np.testing.assert_allclose(to_np(gc)[:, 0], oc, rtol=1e-5, atol=0)
    new_lam = np.stack([to_np(cache.gate(l, X[l][:, None].contiguous())[1])[seq, 0] for l in range(w.layers)])  # [L, H]
    new_c = orc.horizon_term_from_lambda32(new_lam, w.horizon)
    # the library derives c on the device in fp32; the selection is checked on the device's own values
    new_c_dev = np.stack([to_np(cache.gate(l, X[l][:, None].contiguous())[2])[seq, 0] for l in range(w.layers)])
    np.testing.assert_allclose(new_c_dev, new_c, rtol=1e-5, atol=0)

    # ---- attention of the sampled pools: rows before the step plus the new token
    g = w.group
    for (l, h) in set(sample_pools):
        pos, lam, c, kk, vv = before[(l, h)]
        Kp = np.concatenate([kk, to_np(K[l, seq, h])[None].astype(np.float64)])
        Vp = np.concatenate([vv, to_np(V[l, seq, h])[None].astype(np.float64)])
        for j in range(h * g, (h + 1) * g):
            want = orc.attention(to_np(Q[l, seq, j]), Kp, Vp)
            err = np.abs(to_np(out[l, seq, j]) - want).max()
            assert err <= 2e-2, f"attention error {err} in pool ({seq},{l},{h}), head {j}"

    # ---- selection of the sampled sequence: full sort over (old entries + the new token) at time t + 1
    lam_all, c_all, pos_all, lay_all, head_all = [], [], [], [], []
    for l in range(w.layers):
        for h in range(w.kv_heads):
            pos, lam, c, _, _ = before[(l, h)]
            lam_all += [lam, new_lam[l, h:h + 1]]
            c_all += [c, new_c_dev[l, h:h + 1]]
            pos_all += [pos, np.array([t + 1], np.int64)]
            lay_all.append(np.full(len(pos) + 1, l, np.int64))
            head_all.append(np.full(len(pos) + 1, h, np.int64))
    lam_all, c_all, pos_all = np.concatenate(lam_all), np.concatenate(c_all), np.concatenate(pos_all)
    lay_all, head_all = np.concatenate(lay_all), np.concatenate(head_all)
    S = orc.score(lam_all, c_all, pos_all, t + 1)
    keep = orc.select_keep(S, pos_all, lay_all, head_all, w.budget_entries)
    mask = np.zeros(len(S), bool)
    mask[keep] = True
    after_lens = cache.lengths()
    for b in range(w.batch):
        assert int(after_lens[b].sum()) == w.budget_entries           # budget invariant, every sequence
    for l in range(w.layers):
        for h in range(w.kv_heads):
            sel = mask & (lay_all == l) & (head_all == h)
            want = np.sort(pos_all[sel])
            got = cache.kept(seq, l, h, len(want) + 2).numpy()
            np.testing.assert_array_equal(got, want, err_msg=f"kept set differs in pool ({seq},{l},{h})")
    assert (cache.select_stats()[:, 0] == 0).all()                     # the sampled candidate range held
    cache.check_invariants()
    cache.close()


@pytest.mark.parametrize("name,context", [("llama8b_32k", 4608), ("qwen_vl_16k", 2560), ("stress_128k", 8704)])
def test_full_size_chunk_attention_matches_oracle_on_samples(name, context):
    """trimkv_prefill_attention at the full shapes, cache at its budget, chunk of the workload's size: sampled (sequence,
    token, query head) outputs against the oracle's fp64 attention over the entries that token may see (everything kept
    from before the chunk, then the chunk's own tokens up to itself), read back from the device in pool order."""
    w = workloads.WORKLOADS[name]
    seed = 0
    cache = binding.TrimKV.from_workload(w)
    per_layer, w_g = workloads.gate_params(w, seed, device=DEV)
    for l, p in enumerate(per_layer):
        cache.set_gate(l, *p)
    cache.set_shared_projection(w_g, w.b_g)
    bank = workloads.ProjectionBank(w, seed, device=DEV)
    _prefill(cache, w, bank, seed, context)
    rng = np.random.default_rng(11)
    n = w.chunk
    g = w.group
    qs = {}                                              # the chunk goes to every layer; three layers are checked
    for l in range(w.layers):
        x = workloads.hidden_states(w, seed, l, context, n, device=DEV)
        q, k, v = workloads.project_qkv(w, bank, l, x)
        cache.append(l, k, v, x=x)
        if l in (0, w.layers // 2, w.layers - 1):
            qs[l] = (q, cache.prefill_attention(l, q))
    cache.sync_status()
    lens = cache.lengths().numpy()
    for l, (q, out) in qs.items():
        for _ in range(3):
            b, h = int(rng.integers(w.batch)), int(rng.integers(w.kv_heads))
            total = int(lens[b, l, h])
            n_old = total - n
            assert n_old >= 0
            _, _, _, kk, vv = cache.pool(b, l, h, total, with_kv=True)
            kk, vv = to_np(kk).astype(np.float64), to_np(vv).astype(np.float64)
            for j in (0, int(rng.integers(n)), n - 1):
                for hq in (h * g, h * g + int(rng.integers(g))):
                    vis = n_old + j + 1
                    want = orc.attention(to_np(q[b, j, hq]), kk[:vis], vv[:vis])
                    err = np.abs(to_np(out[b, j, hq]) - want).max()
                    assert err <= 2e-2, f"chunk attention error {err} at (seq {b}, layer {l}, token {j}, head {hq})"
    cache.score_and_evict()
    cache.sync_status()
    cache.close()


def _keep_mask_from_words(bits, n):
    """bool [n] on the device from the packed keep words (bit i of word i // 64, little-endian)."""
    b8 = bits.view(torch.uint8)
    m = ((b8[:, None] >> torch.arange(8, device=b8.device, dtype=torch.uint8)[None, :]) & 1).reshape(-1)[:n]
    return m.bool()


@pytest.mark.parametrize("log2n,kind", [(28, "uniform"), (26, "two_values")])
def test_select_topk_properties_at_sweep_sizes(log2n, kind):
    """The standalone selection at the sweep's sizes, where a full sort on the host is out of reach: properties that pin
    the result at any size.  Exactly k entries are kept; no evicted score exceeds a kept one; among entries whose score
    equals the threshold the kept ones are exactly those with the smallest indices (ties keep the older entry)."""
    n = 1 << log2n
    if kind == "uniform":
        s = workloads.selection_scores(n, seed=3, device=DEV)
    else:
        s = (workloads.selection_scores(n, seed=4, device=DEV) > -5.0).float() * 2.0 - 7.0      # -5 or -7, heavy ties
    for k in (n // 8, n - 512):
        bits, status = binding.select_topk(s, k)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        keep = _keep_mask_from_words(bits, n)
        assert int(keep.sum().item()) == k
        tau = s[keep].min()                                   # lowest kept score
        assert float(s[~keep].max().item()) <= float(tau.item())
        tie = s == tau                                        # entries on the threshold: kept ones come first by index
        idx = torch.nonzero(tie, as_tuple=False).reshape(-1)
        kept_tie = keep[idx]
        n_kept_tie = int(kept_tie.sum().item())
        assert bool(kept_tie[:n_kept_tie].all().item()) and not bool(kept_tie[n_kept_tie:].any().item())
        del keep, tie, idx, kept_tie


def test_multi_turn_flow_at_full_shape():
    """The multi-turn workload at its full shape (32 layers, 8 KV heads, batch 32, budget 524,288 entries per sequence),
    two turns: each turn appends 2048 user tokens in 512-token chunks with an eviction round after every chunk (up to
    131,072 evictions per sequence and round) and then decodes 8 tokens through trimkv_decode_step_all; positions and
    the budget persist across the turns.  One sampled sequence is mirrored by the oracle through the whole flow (fed
    the device's fp32 retention terms): pool lengths after every eviction round, the kept set of every one of its pools
    after each turn's prompt and each turn's decode steps, bit for bit; the budget invariant for every sequence; and
    the attention output of sampled pools in each turn's last decode step."""
    w = workloads.WORKLOADS["multiturn"]
    seed, seq = 0, 11
    LH = w.layers * w.kv_heads
    cache = binding.TrimKV.from_workload(w)
    per_layer, w_g = workloads.gate_params(w, seed, device=DEV)
    for l, p in enumerate(per_layer):
        cache.set_gate(l, *p)
    cache.set_shared_projection(w_g, w.b_g)
    bank = workloads.ProjectionBank(w, seed, device=DEV)
    oc = orc.OracleCache(w.budget_entries, w.layers, w.kv_heads, w.q_heads, 0, w.horizon)
    empty = lambda n: np.zeros((n, w.kv_heads, 0))
    rng = np.random.default_rng(3)
    g = w.group

    def check_lengths():
        lens = cache.lengths().numpy()
        np.testing.assert_array_equal(lens[seq], oc.lengths())
        want = min(w.budget_entries, oc.tokens[0] * LH)
        assert (lens.reshape(w.batch, -1).sum(1) == want).all()          # budget invariant, every sequence

    def check_sets():
        for l in range(w.layers):
            for h in range(w.kv_heads):
                want = oc.kept_positions(l, h)
                got = cache.kept(seq, l, h, len(want) + 2).numpy()
                np.testing.assert_array_equal(got, want, err_msg=f"kept set differs in pool ({seq},{l},{h})")

    tokens = 0
    for turn in range(2):
        for ch in range(w.context // w.chunk):
            for l in range(w.layers):
                x = workloads.hidden_states(w, seed, l, tokens, w.chunk, device=DEV)
                _, k, v = workloads.project_qkv(w, bank, l, x)
                cache.append(l, k, v, x=x)
                _, lam, c = cache.gate(l, x)                         # the terms the append computed (same kernels)
                oc.append(l, empty(w.chunk), empty(w.chunk), lam=to_np(lam[seq]), c=to_np(c[seq]))
            cache.score_and_evict()
            oc.score_and_evict()
            tokens += w.chunk
            check_lengths()
        check_sets()
        for step in range(8):
            X, K, V, Q = _step_inputs(w, bank, seed, tokens)
            last = step == 7
            if last:                                                   # sampled pools before the step, with their rows
                pools = [(int(rng.integers(w.layers)), int(rng.integers(w.kv_heads))) for _ in range(3)]
                rows = {}
                for (l, h) in pools:
                    n_old = len(oc.kept_positions(l, h))
                    _, _, _, kk, vv = cache.pool(seq, l, h, n_old + 2, with_kv=True)
                    rows[(l, h)] = (to_np(kk).astype(np.float64), to_np(vv).astype(np.float64))
            out = torch.empty_like(Q)
            cache.decode_step_all(K, V, Q, out, x=X)
            for l in range(w.layers):
                _, lam, c = cache.gate(l, X[l][:, None].contiguous())
                oc.append(l, empty(1), empty(1), lam=to_np(lam[seq]), c=to_np(c[seq]))
            oc.score_and_evict()
            tokens += 1
            check_lengths()
            if last:
                for (l, h), (kk, vv) in rows.items():
                    Kp = np.concatenate([kk, to_np(K[l, seq, h])[None].astype(np.float64)])
                    Vp = np.concatenate([vv, to_np(V[l, seq, h])[None].astype(np.float64)])
                    for j in range(h * g, (h + 1) * g):
                        err = np.abs(to_np(out[l, seq, j]) - orc.attention(to_np(Q[l, seq, j]), Kp, Vp)).max()
                        assert err <= 2e-2, f"attention error {err} in pool ({seq},{l},{h}), head {j}, turn {turn}"
        check_sets()
    # positions kept counting across the turns: the newest kept position is the last token of the second turn
    assert max(int(oc.kept_positions(l, h).max()) for l in range(w.layers) for h in range(w.kv_heads)
               if len(oc.kept_positions(l, h))) == tokens
    assert (cache.select_stats()[:, 0] == 0).all()
    cache.check_invariants()
    cache.close()
