"""The layer-sharded eviction round with the CUDA stages (trimkv_shard_* through the C ABI).  One GPU is enough: every
emulated rank is a handle of its own holding a slice of the layers, the ranks run the exchange protocol on threads of
this process (tests/util_sharded.ThreadComm), and no kernel ever waits for another rank's kernel -- the ranks meet on
the host between stages.  The kept set of every pool must equal what the single-process oracle keeps under the one
global budget, in the normal path and with the exact radix fallback forced."""
import numpy as np
import pytest
import torch

from oracle import trimkv_oracle as orc
from paper_2605_09649_b200 import binding, sharded
from test_sharded_cpu import B, BUDGET, H, L, SCHEDULE, scenario_inputs
from util_sharded import run_ranks_in_threads

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("world,distrust", [(1, False), (2, False), (4, False), (2, True), (4, True)])
def test_sharded_eviction_on_the_gpu_equals_single_process_oracle(world, distrust):
    inputs = scenario_inputs(seed=5)
    oracles = [orc.OracleCache(BUDGET, L, H, H, 0, 2) for _ in range(B)]
    want = []                                                   # per round: kept positions of every pool
    for lam, c in inputs:
        n = lam.shape[2]
        for b in range(B):
            for l in range(L):
                oracles[b].append(l, np.zeros((n, H, 0)), np.zeros((n, H, 0)), lam=lam[l, b], c=c[l, b])
            oracles[b].score_and_evict()
        want.append([[[oracles[b].kept_positions(l, h) for h in range(H)] for l in range(L)] for b in range(B)])
    per = L // world
    fallbacks = [0] * world

    def rank_body(rank, comm):
        torch.cuda.set_device(0)
        l0 = rank * per
        cache = binding.TrimKV(BUDGET, per, H, 128, q_heads=H, batch=B, max_chunk=max(SCHEDULE), shard_total_layers=L,
                               shard_layer0=l0)
        if distrust:
            cache.set_test_hooks(binding.TEST_DISTRUST_SAMPLE)
        stages = sharded.CudaStages(cache)
        held = 0
        for rnd, (lam, c) in enumerate(inputs):
            n = lam.shape[2]
            k = torch.zeros(B, n, H, 128, device=DEV, dtype=torch.bfloat16)
            for l in range(per):
                cache.append(l, k, k, lam=torch.from_numpy(lam[l0 + l]).to(DEV), c=torch.from_numpy(c[l0 + l]).to(DEV))
            n_total = held + n * L * H
            info = sharded.sharded_evict(stages, comm, n_total, n_total - BUDGET)
            fallbacks[rank] += int(info["fallback"])
            held = BUDGET
            total = comm.all_gather(torch.tensor(info["local_entries"], dtype=torch.int64))
            assert (total.sum(0) == BUDGET).all()
            for b in range(B):
                for l in range(per):
                    for h in range(H):
                        got = cache.kept(b, l, h, 4096).numpy()
                        np.testing.assert_array_equal(got, want[rnd][b][l0 + l][h], err_msg=f"round {rnd} pool ({b},{l0 + l},{h})")
        cache.check_invariants()
        cache.close()

    run_ranks_in_threads(world, rank_body)
    assert all(f == (len(SCHEDULE) if distrust else 0) for f in fallbacks), fallbacks


def test_sharded_handle_refuses_the_single_handle_eviction_calls():
    cache = binding.TrimKV(64, 2, 1, 128, batch=1, max_chunk=8, shard_total_layers=4, shard_layer0=2)
    with pytest.raises(binding.TrimkvError) as e:
        cache.score_and_evict()
    assert e.value.status == binding.E_STATE
    plain = binding.TrimKV(64, 2, 1, 128, batch=1, max_chunk=8)
    with pytest.raises(binding.TrimkvError):
        sharded.CudaStages(plain).filter()
    cache.close(); plain.close()


def test_sharded_eviction_at_the_llama_shape_equals_the_single_handle_run():
    """Full shape (32 layers, 8 KV heads, batch 8, global budget 1,048,576 entries per sequence), two emulated ranks of 16
    layers each: 512-token chunks (131,072 evictions per sequence and round once the budget is full: candidate exchanges
    of ~10^5 records) and single-token decode steps.  The single-handle run of the same inputs is the reference (it is
    checked against the oracle at this shape in test_gpu_fullsize.py): pool lengths of every sequence and the kept set
    of every pool of a sampled sequence must be identical, decode attention within tolerance."""
    from paper_2605_09649_b200 import workloads
    w = workloads.WORKLOADS["llama8b_32k"]
    seed, seq, world, context, steps = 0, 6, 2, 4608, 3
    LH = w.layers * w.kv_heads
    per_layer, w_g = workloads.gate_params(w, seed, device=DEV)
    bank = workloads.ProjectionBank(w, seed, device=DEV)

    def feed(cache, l_global, l_local, off, n, attend):
        x = workloads.hidden_states(w, seed, l_global, off, n, device=DEV)
        q, k, v = workloads.project_qkv(w, bank, l_global, x)
        cache.append(l_local, k, v, x=x)
        return cache.decode_attention(l_local, q[:, -1].contiguous()) if attend else None

    def setup(cache, l0, nl):
        for l in range(nl):
            cache.set_gate(l, *per_layer[l0 + l])
        cache.set_shared_projection(w_g, w.b_g)

    # ---- reference: one handle holds all layers
    ref = binding.TrimKV.from_workload(w)
    setup(ref, 0, w.layers)
    ref_out = []
    for off in range(0, context, w.chunk):
        for l in range(w.layers):
            feed(ref, l, l, off, w.chunk, False)
        ref.score_and_evict()
    for i in range(steps):
        ref_out.append(torch.stack([feed(ref, l, l, context + i, 1, True) for l in range(w.layers)]))
        ref.score_and_evict()
    ref_lens = ref.lengths()
    ref_kept = {(l, h): ref.kept(seq, l, h, int(ref_lens[seq, l, h]) + 1) for l in range(w.layers) for h in range(w.kv_heads)}
    ref.close()

    per = w.layers // world
    results = [None] * world

    def rank_body(rank, comm):
        torch.cuda.set_device(0)
        l0 = rank * per
        cache = binding.TrimKV.from_workload(w.replace(layers=per), shard_total_layers=w.layers, shard_layer0=l0)
        setup(cache, l0, per)
        stages = sharded.CudaStages(cache)
        held, outs, cands = 0, [], []

        def evict(n):
            nonlocal held
            n_total = held + n * LH
            if n_total > w.budget_entries:
                info = sharded.sharded_evict(stages, comm, n_total, n_total - w.budget_entries)
                assert not info["fallback"]
                cands.append(info["candidates"])
                held = w.budget_entries
            else:
                held = n_total

        for off in range(0, context, w.chunk):
            for l in range(per):
                feed(cache, l0 + l, l, off, w.chunk, False)
            evict(w.chunk)
        for i in range(steps):
            outs.append(torch.stack([feed(cache, l0 + l, l, context + i, 1, True) for l in range(per)]))
            evict(1)
        cache.check_invariants()
        lens = cache.lengths()
        kept = {(l0 + l, h): cache.kept(seq, l, h, int(lens[seq, l, h]) + 1) for l in range(per) for h in range(w.kv_heads)}
        results[rank] = (lens, kept, outs, cands)
        cache.close()

    run_ranks_in_threads(world, rank_body)
    lens = torch.cat([results[r][0] for r in range(world)], dim=1)
    assert torch.equal(lens, ref_lens)
    assert (lens.reshape(w.batch, -1).sum(1) == w.budget_entries).all()
    for r in range(world):
        for key, got in results[r][1].items():
            assert torch.equal(got, ref_kept[key]), key
    for i in range(steps):
        got = torch.cat([results[r][2][i] for r in range(world)], dim=0)
        assert float((got.float() - ref_out[i].float()).abs().max()) <= 2e-2
    assert max(results[0][3]) > 10000                       # the chunk rounds really exchanged large candidate lists
