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
CASES = [("llama8b_32k", 32768, 0), ("qwen_vl_16k", 4096, 2), ("stress_128k", 9216, 0), ("multiturn", 2048, 5)]


@pytest.mark.parametrize("name,context,seq", CASES)
def test_full_size_step_matches_oracle_on_samples(name, context, seq):
    w = workloads.WORKLOADS[name]
    seed = 0
    LH = w.layers * w.kv_heads
    cache = binding.TrimKV.from_workload(w)
    per_layer, w_g = workloads.gate_params(w, seed, device=DEV)
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
