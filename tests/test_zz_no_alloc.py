"""The allocation-free selection entry point against the context-based path.

`cake_select_positions_static` serves callers that may not allocate device memory at call
time (code inside another framework's memory plan, latency-critical serving loops): its
scratch is a fixed array inside the library.  Here its output is compared, bit for bit as for
every index result in this suite, with what the ordinary entry points (cake_set_indicators ->
cake_allocate -> cake_evict -> cake_get_positions on a one-layer context) select from the
same values, on two calls in a row so that the second one meets the first one's leftovers in
the shared scratch.  This file sorts last on purpose: a run that stops at the first failure
has then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import cake_oracle as O
from paper_2503_12491_b200 import binding
from paper_2503_12491_b200.binding import Cake, CakeError, CAKE_ERR_ARG, CAKE_ERR_CAPACITY

pytestmark = pytest.mark.gpu

WINDOW = 4


def positions_via_context(values: torch.Tensor, keep: int) -> torch.Tensor:
    """The same selection through a one-layer context: the first `keep` retained positions."""
    n_heads, n = values.shape
    N = n + WINDOW
    cake = Cake(n_layers=1, n_q_heads=n_heads, n_kv_heads=n_heads, head_dim=64, window=WINDOW,
                pool_kernel=1, gamma=0.0, total_budget=WINDOW + keep, max_requests=1,
                max_total_tokens=N, dtype=torch.float32)
    cake.begin([0, N])
    full = torch.zeros(n_heads, N, dtype=torch.float32, device="cuda")
    full[:, :n] = values
    cake.set_preferences(torch.ones(1, 1, dtype=torch.float64, device="cuda"))
    cake.set_indicators(0, full)
    cake.allocate(0)
    cake.evict(0)
    got = cake.get_positions(0, 0, keep + WINDOW)[:, :keep].clone()
    assert cake.status() == 0
    cake.destroy()
    return got


def test_static_selection_matches_context_path_twice_in_a_row():
    g = torch.Generator(device="cuda").manual_seed(1234)
    cases = [(6, 5000, 1300), (3, 777, 400)]       # second call: smaller, other tie pattern
    for call, (heads, n, keep) in enumerate(cases):
        vals = torch.randn(heads, n, generator=g, device="cuda")
        if call == 1:
            vals = torch.round(vals * 2) / 2       # many exact ties across the threshold
        vals[0, :] = 0.25                          # one head entirely tied: lowest positions win
        out = torch.full((heads, keep), -1, dtype=torch.int32, device="cuda")
        binding.select_positions_static(vals, keep, out=out)
        want = positions_via_context(vals, keep)
        torch.cuda.synchronize()
        assert torch.equal(out, want), f"call {call}"
        assert torch.equal(out[0].cpu(), torch.arange(keep, dtype=torch.int32))
        # and against the oracle's TopK of Eq. 12: value descending, position ascending
        v = vals.cpu().numpy().astype(np.float64)
        for h in range(heads):
            assert np.array_equal(out[h].cpu().numpy(), O.topk_keep(v[h], keep))


def test_static_selection_rejects_what_does_not_fit():
    lib = binding.load_library()
    vals = torch.zeros(1, 64, dtype=torch.float32, device="cuda")
    out = torch.zeros(1, 64, dtype=torch.int32, device="cuda")
    # 33 heads of 32768 values need 33792 bitmap words: one more than the built-in scratch holds
    rc = lib.cake_select_positions_static(vals.data_ptr(), 33, 32768, 8, out.data_ptr(), None)
    assert rc == CAKE_ERR_CAPACITY
    assert lib.cake_select_positions_static(vals.data_ptr(), 1, 64, 65, out.data_ptr(), None) == CAKE_ERR_ARG
    with pytest.raises(CakeError):
        binding.select_positions_static(vals, 65, out=out)
    # edge sizes: keep everything, keep nothing
    binding.select_positions_static(vals, 64, out=out)
    assert torch.equal(out[0].cpu(), torch.arange(64, dtype=torch.int32))
    assert binding.select_positions_static(vals, 0).shape == (1, 0)
