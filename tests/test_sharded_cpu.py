"""The layer-sharded eviction round on CPU ranks (gloo, world 2 and 4): every rank holds a slice of the layers, runs the
exchange protocol of paper_2605_09649_b200/sharded.py around a numpy statement of the rank-local stages
(tests/util_sharded.HostStages), and the kept set of every pool must equal what the single-process oracle keeps when it
ranks ALL layers and heads under the one global budget (Sec. 4.2) -- in the normal path and when the sampled bracket
misses and the exact radix fallback decides."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import trimkv_oracle as orc
from paper_2605_09649_b200 import sharded
from util_sharded import HostStages

L, H, B, BUDGET = 8, 2, 2, 700
SCHEDULE = [300, 150, 1, 1, 40, 1]            # tokens appended per round (a round = append to every layer, then evict)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def scenario_inputs(seed):
    """Per round: lam, c [L, B, n, H] fp32 (identical on every rank: same seed)."""
    r = np.random.default_rng(seed)
    out = []
    for i, n in enumerate(SCHEDULE):
        if i % 2 == 0:
            lam = -np.abs(r.normal(0, 0.05, size=(L, B, n, H))).astype(np.float32)
        else:                                  # heavy ties: few distinct retention values
            vals = -np.abs(r.normal(0, 0.05, size=4)).astype(np.float32)
            lam = vals[r.integers(0, 4, size=(L, B, n, H))]
        lam *= (1.0 + 3.0 * r.random((L, 1, 1, H))).astype(np.float32)         # layers and heads differ: ragged pools
        out.append((lam, orc.horizon_term_from_lambda32(lam, 2)))
    return out


def run_rank(rank, world, comm, distrust, seed=3):
    per = L // world
    l0 = rank * per
    st = HostStages(rank, l0, per, L, H, B, distrust=distrust)
    oracles = [orc.OracleCache(BUDGET, L, H, H, 0, 2) for _ in range(B)]
    held = 0
    fallbacks = 0
    for lam, c in scenario_inputs(seed):
        n = lam.shape[2]
        st.append_token_block(lam[l0:l0 + per], c[l0:l0 + per])
        for b in range(B):
            for l in range(L):
                oracles[b].append(l, np.zeros((n, H, 0)), np.zeros((n, H, 0)), lam=lam[l, b], c=c[l, b])
        n_total = held + n * L * H
        k = n_total - BUDGET
        if k > 0:
            info = sharded.sharded_evict(st, comm, n_total, k)
            fallbacks += int(info["fallback"])
            held = BUDGET
            g = comm.all_gather(torch.tensor(info["local_entries"], dtype=torch.int64))
            assert (g.sum(0) == BUDGET).all()                                    # budget invariant over all ranks
        else:
            held = n_total
        for b in range(B):
            oracles[b].score_and_evict()
            for l in range(l0, l0 + per):
                for h in range(H):
                    np.testing.assert_array_equal(st.kept_positions(b, l, h), oracles[b].kept_positions(l, h),
                                                  err_msg=f"rank {rank} pool ({b},{l},{h})")
    return fallbacks


def _worker(rank, world, port, distrust, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        fb = run_rank(rank, world, sharded.TorchComm(), distrust)
        q.put((rank, "ok", fb))
    except BaseException as e:      # noqa: BLE001
        q.put((rank, repr(e), 0))
        raise
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,distrust", [(2, False), (4, False), (2, True), (4, True)])
def test_sharded_eviction_equals_single_process_oracle(world, distrust):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, distrust, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=240) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert all(r[1] == "ok" for r in res), res
    rounds_with_eviction = len(SCHEDULE)                         # every round exceeds the budget
    if distrust:
        assert all(r[2] == rounds_with_eviction for r in res)        # the exact fallback decided every round
    else:
        assert all(r[2] == 0 for r in res)                           # the sampled bracket held every time


def test_eviction_keys_order_is_the_oracles_total_order():
    """The 64-bit keys the host stages rank by: ascending key order = the reverse of the oracle's keep order."""
    from util_sharded import eviction_keys, pool_bits_of
    r = np.random.default_rng(0)
    n = 500
    S = r.choice(np.array([-1.5, -0.25, 0.0, -0.0, 3.0, -np.inf], np.float32), size=n)
    pos = r.integers(1, 50, size=n)
    layer, head = r.integers(0, 4, size=n), r.integers(0, 2, size=n)
    # make (pos, layer, head) unique so that the order is total
    _, first = np.unique(np.stack([pos, layer, head]), axis=1, return_index=True)
    S, pos, layer, head = S[first], pos[first], layer[first], head[first]
    keys = eviction_keys(S, pos, layer * 2 + head, pool_bits_of(8))
    assert len(np.unique(keys)) == len(keys)
    for budget in (1, len(S) // 3, len(S) - 1):
        keep = orc.select_keep(S, pos, layer, head, budget)
        by_key = np.sort(np.argsort(keys)[len(S) - budget:])
        np.testing.assert_array_equal(by_key, keep)
