"""Parity of every exposed `cake_config` option and kernel instantiation against the oracle,
on small cases that still span several key tiles and a ragged tail: pooling mode and kernel
size, variance divisor, temperatures, head_dim 64 on the tensor-core path, grouped-query
factors 2 and 8, and the mode in which the caller supplies the window rows' log-sum-exps."""
import numpy as np
import pytest
import torch

from oracle import cake_oracle as O
from paper_2503_12491_b200 import synth, harness
from paper_2503_12491_b200.binding import CAKE_POOL_AVG, CAKE_POOL_MAX

pytestmark = pytest.mark.gpu

RTOL = 1e-3


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def assert_close(got, want, what, rtol=RTOL):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    bad = err > rtol * np.abs(want) + 1e-30
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} beyond rtol {rtol}; "
                           f"worst rel {np.max(err / (np.abs(want) + 1e-300)):.3e}")


def bf16_case(**kw):
    base = dict(n_layers=2, n_q_heads=8, n_kv_heads=2, seq_lens=(1333, 417), total_budget=2 * 160)
    base.update(kw)
    return synth.scaled(synth.workload(3), **base)


def fp32_case(**kw):
    base = dict(n_layers=2, seq_lens=(700, 129), total_budget=2 * 90)
    base.update(kw)
    return synth.scaled(synth.workload(1), **base)


def check_scores(w, *, cake_kw=None, oracle_kw=None, expect_tc=None, lse=False):
    """Scores every layer through the C-ABI and compares indicators, H, V, P with the oracle
    called with the matching options."""
    cake_kw, oracle_kw = cake_kw or {}, oracle_kw or {}
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w, **cake_kw)
    if expect_tc is not None:
        assert cake.uses_tensor_cores() == expect_tc
    cake.begin(w.cu_seqlens)
    cu = w.cu_seqlens
    refs = []
    for l in range(w.n_layers):
        supplied = None
        if lse:
            supplied = torch.empty(len(w.seq_lens), w.n_q_heads, w.window, dtype=torch.float32,
                                   device="cuda")
            for r, N in enumerate(w.seq_lens):
                s = O.window_logits(to_np(qs[l][r]), to_np(ks[l][:, cu[r]:cu[r + 1]]))
                m = s.max(axis=-1, keepdims=True)
                supplied[r] = torch.from_numpy(
                    (m[..., 0] + np.log(np.exp(s - m).sum(axis=-1))).astype(np.float32)).cuda()
        cake.score_layer(l, qs[l], ks[l], lse=supplied)
        ind = cake.get_indicators(l).cpu().numpy()
        per = []
        for r, N in enumerate(w.seq_lens):
            n = N - w.window
            ref = O.score_layer(to_np(qs[l][r]), to_np(ks[l][:, cu[r]:cu[r + 1]]), gamma=w.gamma,
                                pool_kernel=w.pool_kernel, tau1=w.tau1, tau2=w.tau2, **oracle_kw)
            assert_close(ind[:, cu[r]:cu[r] + n], ref["indicator"], f"indicator l{l} r{r}")
            assert np.all(np.isinf(ind[:, cu[r] + n:cu[r + 1]]))
            per.append(ref)
        refs.append(per)
        cake.allocate(l)
        cake.evict(l)
    H, V, P = (x.cpu().numpy() for x in cake.get_preferences())
    for l in range(w.n_layers):
        for r in range(len(w.seq_lens)):
            assert_close(H[r, l], refs[l][r]["H"], f"H l{l} r{r}")
            assert_close(V[r, l], refs[l][r]["V"], f"V l{l} r{r}")
            assert_close(P[r, l], refs[l][r]["P"], f"P l{l} r{r}")
    assert cake.status() == 0
    cake.destroy()


@pytest.mark.parametrize("kernel", [1, 3, 5, 7, 9, 13])
@pytest.mark.parametrize("mode,name", [(CAKE_POOL_MAX, "max"), (CAKE_POOL_AVG, "avg")])
def test_pooling_modes_and_kernel_sizes(kernel, mode, name):
    """Section 4.3 pooling: both modes, the unrolled kernels (1..7) and the generic one (>= 9)."""
    w = bf16_case(pool_kernel=kernel, n_layers=1, total_budget=160)
    check_scores(w, cake_kw=dict(pool_mode=mode), oracle_kw=dict(pool_mode=name), expect_tc=True)


@pytest.mark.parametrize("make,tc", [(bf16_case, True), (fp32_case, False)])
def test_unbiased_variance(make, tc):
    """var_ddof = 1 (Eq. 5 and Eq. 11 with the S_w - 1 divisor) on both score paths."""
    check_scores(make(), cake_kw=dict(var_ddof=1), oracle_kw=dict(ddof=1), expect_tc=tc)


@pytest.mark.parametrize("make,tc", [(bf16_case, True), (fp32_case, False)])
def test_temperatures_of_the_preference(make, tc):
    """Eq. 6 with tau1 = 0.5, tau2 = 2."""
    check_scores(make(tau1=0.5, tau2=2.0), expect_tc=tc)


def test_head_dim_64_on_the_tensor_core_path():
    check_scores(bf16_case(head_dim=64), expect_tc=True)


@pytest.mark.parametrize("hq,hkv,window", [(4, 2, 32), (4, 2, 16), (16, 2, 16), (8, 1, 8), (3, 3, 96)])
def test_group_factors_and_row_counts(hq, hkv, window):
    """G = 2 and G = 8 instantiations and tiles of 32, 64, 96 and 128 rows."""
    w = bf16_case(n_q_heads=hq, n_kv_heads=hkv, window=window, total_budget=2 * (window + 100),
                  seq_lens=(1100, 300))
    check_scores(w, expect_tc=True)


@pytest.mark.parametrize("make,tc", [(bf16_case, True), (fp32_case, False)])
def test_supplied_log_sum_exps_give_the_same_preferences(make, tc):
    """With `lse` the row pass is skipped and the entropy comes from the column pass: indicators,
    H, V and P of every layer against the oracle."""
    check_scores(make(n_layers=3, total_budget=3 * 120), expect_tc=tc, lse=True)


def test_supplied_log_sum_exps_grouped_by_eight():
    check_scores(bf16_case(n_q_heads=16, n_kv_heads=2, window=16, total_budget=2 * 120), expect_tc=True,
                 lse=True)


def test_set_preferences_is_refused_once_a_layer_is_evicted():
    from paper_2503_12491_b200.binding import CakeError, CAKE_ERR_STATE
    w = fp32_case()
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    cake.score_layer(0, qs[0], ks[0])
    cake.allocate(0)
    cake.evict(0)
    with pytest.raises(CakeError) as e:
        cake.set_preferences(torch.ones(len(w.seq_lens), 2, dtype=torch.float64, device="cuda"))
    assert e.value.code == CAKE_ERR_STATE
    cake.destroy()


def test_a_refused_begin_does_not_disturb_the_context():
    """A batch that exceeds the capacity is refused; the next batch in the same context gives the
    same bits as before."""
    from paper_2503_12491_b200.binding import CakeError, CAKE_ERR_STATE, CAKE_ERR_CAPACITY
    w = bf16_case()
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    first = cake.run(qs, ks, vs, w.cu_seqlens)[3].clone()
    with pytest.raises(CakeError) as e:
        cake.begin([0, 100000])
    assert e.value.code == CAKE_ERR_CAPACITY
    again = cake.run(qs, ks, vs, w.cu_seqlens)[3]
    assert torch.equal(first, again) and cake.status() == 0
    cake.destroy()


def test_a_wait_that_runs_out_returns_a_status_and_the_context_recovers():
    """Every wait inside the score kernel is bounded.  With a short limit and a launch count that
    no partial result can match (the test hook), the cross-CTA waits run out: the launch returns,
    the device status reads CAKE_ERR_TIMEOUT, and the next batch in the same context is correct."""
    from paper_2503_12491_b200.binding import CAKE_ERR_TIMEOUT
    w = bf16_case()
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    assert cake.uses_tensor_cores()
    want = [t.clone() for t in cake.run(qs, ks, vs, w.cu_seqlens)]
    assert cake.status() == 0
    cake.set_wait_limit(2_000_000)                    # about a millisecond
    cake.begin(w.cu_seqlens)
    cake.debug_skew_sync(1)
    cake.score_layer(0, qs[0], ks[0])
    torch.cuda.synchronize()
    assert cake.status() == CAKE_ERR_TIMEOUT
    cake.set_wait_limit(0)
    got = cake.run(qs, ks, vs, w.cu_seqlens)           # cake_begin clears the status and the hook
    assert cake.status() == 0
    n = int(want[2][-1])
    assert torch.equal(got[2], want[2]) and torch.equal(got[3][:n], want[3][:n])
    assert torch.equal(got[0][:n], want[0][:n]) and torch.equal(got[1][:n], want[1][:n])
    cake.destroy()


# ------------------------------------------------ variants of the paper's comparison study
@pytest.mark.parametrize("make,tc", [(bf16_case, True), (fp32_case, False)])
def test_window_sum_indicator(make, tc):
    """The SnapKV indicator (sum of the window queries' attention) under the preference
    allocation (Section 5.3, compatibility study)."""
    check_scores(make(), cake_kw=dict(indicator_mode=4), oracle_kw=dict(indicator="sum"), expect_tc=tc)


@pytest.mark.parametrize("mode,name,slope", [(1, "uniform", 0.0), (2, "pyramid", 0.6), (2, "pyramid", 1.0)])
def test_uniform_and_pyramid_allocation_bit_exact(mode, name, slope):
    """The fixed allocation patterns of the allocation ablation (Section 5.3) through the same
    rounding, cap and cascade: budgets of every stage and the final retained sets."""
    L = 6
    w = fp32_case(n_layers=L, seq_lens=(400, 90), total_budget=L * 16 + 333)
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w, alloc_mode=mode, pyramid_slope=slope)
    cake.begin(w.cu_seqlens)
    cu = w.cu_seqlens
    inds = []
    for l in range(L):
        cake.score_layer(l, qs[l], ks[l])
        inds.append(cake.get_indicators(l).cpu().numpy())
        cake.allocate(l)
        got = cake.get_budgets().cpu().numpy()
        for r, N in enumerate(w.seq_lens):
            wts = O.allocation_weights([0.0] * (l + 1), L, name, slope)
            want = O.stage_budgets(wts, w.total_budget, L, w.window, N) + w.window
            assert np.array_equal(got[r, :l + 1], want), (l, r, got[r], want)
        cake.evict(l)
    budgets = cake.get_budgets().cpu().numpy()
    for r, N in enumerate(w.seq_lens):
        n = N - w.window
        wts = O.allocation_weights([0.0] * L, L, name, slope)
        c = O.cascade([inds[l][:, cu[r]:cu[r] + n].astype(np.float64) for l in range(L)], wts,
                      total_budget=w.total_budget, window=w.window, seq_len=N)
        assert np.array_equal(budgets[r], c.budgets)
        for l in range(L):
            got_pos = cake.get_positions(r, l, int(budgets[r, l])).cpu().numpy()
            for g in range(w.n_kv_heads):
                assert np.array_equal(got_pos[g], c.positions[l][g])
    assert cake.status() == 0
    cake.destroy()


def test_cumulative_attention_indicator_through_the_hook():
    """H2O's cumulative attention needs the whole prefill attention, which the window-score path
    does not compute: a caller that has it hands it over with cake_set_indicators and gets the
    preference allocation and the cascade on it (Section 5.3, compatibility study)."""
    L = 3
    w = fp32_case(n_layers=L, seq_lens=(260,), total_budget=L * 16 + 150)
    qs, ks, vs = harness.device_inputs(w)
    N, n = w.seq_lens[0], w.seq_lens[0] - w.window
    rng = np.random.default_rng(9)
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    P = np.array([[1.5, 0.4, 2.2]])
    cake.set_preferences(torch.from_numpy(P).cuda())
    inds = []
    for l in range(L):
        q_all = rng.normal(size=(w.n_q_heads, N, w.head_dim))     # stands in for the prompt's queries
        ind = O.cumulative_attention(q_all, to_np(ks[l]))[:, :N].astype(np.float32)
        inds.append(ind)
        cake.set_indicators(l, torch.from_numpy(ind).cuda())
        cake.allocate(l)
        cake.evict(l)
    budgets = cake.get_budgets().cpu().numpy()
    c = O.cascade([x[:, :n].astype(np.float64) for x in inds], P[0], total_budget=w.total_budget,
                  window=w.window, seq_len=N)
    assert np.array_equal(budgets[0], c.budgets)
    for l in range(L):
        got = cake.get_positions(0, l, int(budgets[0, l])).cpu().numpy()
        for g in range(w.n_kv_heads):
            assert np.array_equal(got[g], c.positions[l][g])
    cake.destroy()
