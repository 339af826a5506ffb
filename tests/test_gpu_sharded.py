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
