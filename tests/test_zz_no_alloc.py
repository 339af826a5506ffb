"""trimkv_select_topk_static: the selection for callers that cannot allocate device memory at call time
(fixed memory plans, frameworks that forbid cudaMalloc after start-up).  Its scratch is an array inside
the library, shared by all calls, so the checks here run it twice in a row on different inputs and compare
each result, bit for bit, with trimkv_select_topk (which takes the scratch from the caller).

Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import trimkv_oracle as orc
from paper_2605_09649_b200 import binding, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _both(scores, k):
    n = scores.numel()
    words = max((n + 63) // 64, 1)
    bits = torch.zeros(words, dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.select_topk_static(scores, k, bits, status)
    ref_bits, ref_status = binding.select_topk(scores, k)
    torch.cuda.synchronize()
    return bits.cpu().numpy(), int(status.item()), ref_bits.cpu().numpy(), int(ref_status.item())


def test_static_scratch_selection_equals_workspace_selection_twice_in_a_row():
    # first call: many candidates near the threshold (heavy ties); second call: a different size and
    # distribution, so anything the first call left in the shared scratch would show
    n1, n2 = (1 << 20) + 77, 300_001
    s1 = (workloads.selection_scores(n1, seed=5, device=DEV) * 4).round() / 4
    s2 = workloads.selection_scores(n2, seed=6, device=DEV)
    for scores, k in ((s1, n1 // 3), (s2, n2 - 512), (s1, 1), (s2, n2 // 2)):
        got, st, want, st_ref = _both(scores, k)
        assert st == 0 and st_ref == 0
        np.testing.assert_array_equal(got, want)
        assert int(np.unpackbits(got.view(np.uint8)).sum()) == k


def test_static_scratch_selection_edge_sizes_and_limit():
    s = workloads.selection_scores(1000, seed=7, device=DEV)
    for k in (0, 1000, 2000):
        got, st, want, _ = _both(s, k)
        assert st == 0
        np.testing.assert_array_equal(got, want)
    # beyond the built-in array's limit: refused with a clear message, nothing launched
    big = torch.empty(binding.SELECT_STATIC_MAX_N + 1, dtype=torch.float32, device=DEV)
    bits = torch.zeros((big.numel() + 63) // 64, dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(binding.TrimkvError) as e:
        binding.select_topk_static(big, 10, bits, status)
    assert e.value.status == binding.E_UNSUPPORTED and "limit" in str(e.value)
    # at the limit itself it runs
    at = workloads.selection_scores(binding.SELECT_STATIC_MAX_N, seed=8, device=DEV)
    got, st, want, _ = _both(at, binding.SELECT_STATIC_MAX_N // 8)
    assert st == 0
    np.testing.assert_array_equal(got, want)


def test_static_scratch_selection_matches_the_oracle_and_allocates_nothing():
    """Independent of the sibling entry point: the kept set equals the oracle's full sort (score descending, lower
    index first among equals), and a warmed-up call leaves the device's free memory where it was."""
    n = 300_001
    s = (workloads.selection_scores(n, seed=9, device=DEV) * 8).round() / 8          # heavy ties
    bits = torch.zeros((n + 63) // 64, dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.select_topk_static(s, n // 3, bits, status)                               # warm-up (first call: set-up)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for k in (n // 3, n - 512, 77):
        binding.select_topk_static(s, k, bits, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = np.unpackbits(bits.cpu().numpy().view(np.uint8), bitorder="little")[:n].astype(bool)
        z = np.zeros(n, np.int64)
        want = np.zeros(n, bool)
        want[orc.select_keep(s.cpu().numpy(), np.arange(n), z, z, k)] = True
        np.testing.assert_array_equal(got, want)
    assert torch.cuda.mem_get_info()[0] == free0
