"""Parity of the CUDA path (through the C-ABI) against the CPU oracle.

Tolerances (bf16 or fp32 inputs, fp32 accumulation on the device, float64 in
the oracle): indicators, H, V, P within 1e-3 relative; budgets bit-exact when
the allocator is fed the oracle's preferences; positions and compacted rows
bit-exact when the selection runs on the oracle's indicators; on the device's
own indicators the selected sets may differ from the oracle's only at keys
whose indicator lies within 1e-3 (relative) of the k-th value.
"""
import numpy as np
import pytest
import torch

from oracle import cake_oracle as O
from paper_2503_12491_b200 import synth, harness
from paper_2503_12491_b200.binding import CakeError, CAKE_ERR_STATE, CAKE_ERR_ARG, CAKE_ERR_CAPACITY

pytestmark = pytest.mark.gpu

RTOL = 1e-3


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64) if t.dtype != torch.float64 \
        else t.detach().cpu().numpy()


def oracle_scores(w, qs, ks):
    """Per layer, per request: the oracle's score_layer on the same inputs."""
    cu = w.cu_seqlens
    out = []
    for l in range(len(qs)):
        per = []
        for r in range(len(w.seq_lens)):
            q = to_np(qs[l][r])
            k = to_np(ks[l][:, cu[r]:cu[r + 1]])
            per.append(O.score_layer(q, k, gamma=w.gamma, pool_kernel=w.pool_kernel,
                                     tau1=w.tau1, tau2=w.tau2))
        out.append(per)
    return out


def assert_close(got, want, what, rtol=RTOL):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    tol = rtol * np.abs(want) + 1e-30
    bad = err > tol
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} beyond rtol {rtol}; "
                           f"worst rel {np.max(err / (np.abs(want) + 1e-300)):.3e}")


SMALL_CASES = {
    "tiny-fp32": lambda: synth.workload(1),
    "mha-bf16": lambda: synth.scaled(synth.workload(2), n_layers=3, n_q_heads=4, n_kv_heads=4,
                                     seq_lens=(1500,), total_budget=3 * 200),
    "gqa-bf16": lambda: synth.scaled(synth.workload(3), n_layers=3, n_q_heads=8, n_kv_heads=2,
                                     seq_lens=(2311,), total_budget=3 * 300),
    "gqa-needles": lambda: synth.scaled(synth.workload(4), n_layers=2, n_q_heads=8, n_kv_heads=2,
                                        seq_lens=(3000,), total_budget=2 * 256),
    "ragged": lambda: synth.scaled(synth.workload(5), n_layers=3, n_q_heads=8, n_kv_heads=2,
                                   seq_lens=(700, 129, 1031, 64), total_budget=3 * 128),
    "fp32-d128-avgless": lambda: synth.scaled(synth.workload(1), head_dim=128, n_q_heads=8,
                                              n_kv_heads=4, seq_lens=(333, 200), window=8),
}


@pytest.fixture(scope="module", params=list(SMALL_CASES))
def case(request):
    w = SMALL_CASES[request.param]()
    qs, ks, vs = harness.device_inputs(w)
    return w, qs, ks, vs, oracle_scores(w, qs, ks)


def test_score_layer_matches_oracle(case):
    w, qs, ks, vs, ref = case
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    cu = w.cu_seqlens
    for l in range(w.n_layers):
        cake.score_layer(l, qs[l], ks[l])
        ind = cake.get_indicators(l).cpu().numpy()
        for r, N in enumerate(w.seq_lens):
            n = N - w.window
            assert_close(ind[:, cu[r]:cu[r] + n], ref[l][r]["indicator"], f"indicator l{l} r{r}")
            assert np.all(np.isinf(ind[:, cu[r] + n:cu[r + 1]]))
        cake.allocate(l)
        cake.evict(l)
    H, V, P = (x.cpu().numpy() for x in cake.get_preferences())
    for l in range(w.n_layers):
        for r in range(len(w.seq_lens)):
            assert_close(H[r, l], ref[l][r]["H"], f"H l{l} r{r}")
            assert_close(V[r, l], ref[l][r]["V"], f"V l{l} r{r}")
            assert_close(P[r, l], ref[l][r]["P"], f"P l{l} r{r}")
    assert cake.status() == 0
    cake.destroy()


def test_score_layer_with_supplied_lse(case):
    w, qs, ks, vs, ref = case
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    cu = w.cu_seqlens
    # natural-log LSE of every window row over its visible keys, from torch in fp32
    lse = torch.empty(len(w.seq_lens), w.n_q_heads, w.window, dtype=torch.float32, device="cuda")
    for r, N in enumerate(w.seq_lens):
        q = qs[0][r].float()
        k = ks[0][:, cu[r]:cu[r + 1]].float().repeat_interleave(w.group, dim=0)
        s = torch.einsum("hid,hjd->hij", q, k) / (w.head_dim ** 0.5)
        i = torch.arange(w.window, device="cuda")[:, None]
        j = torch.arange(N, device="cuda")[None, :]
        s = s.masked_fill(j > (N - w.window) + i, float("-inf"))
        lse[r] = torch.logsumexp(s.double(), dim=-1).float()
    cake.score_layer(0, qs[0], ks[0], lse=lse)
    ind = cake.get_indicators(0).cpu().numpy()
    for r, N in enumerate(w.seq_lens):
        n = N - w.window
        assert_close(ind[:, cu[r]:cu[r] + n], ref[0][r]["indicator"], f"indicator (lse) r{r}")
    cake.destroy()


def test_allocator_is_bit_exact_on_oracle_preferences(case):
    w, qs, ks, vs, ref = case
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    R, L = len(w.seq_lens), w.n_layers
    P = np.array([[ref[l][r]["P"] for l in range(L)] for r in range(R)], dtype=np.float64)
    cake.set_preferences(torch.from_numpy(P).cuda())
    for m in range(L):
        cake.allocate(m)
        got = cake.get_budgets().cpu().numpy()
        for r, N in enumerate(w.seq_lens):
            want = O.stage_budgets(P[r, :m + 1], w.total_budget, L, w.window, N) + w.window
            assert np.array_equal(got[r, :m + 1], want), (m, r, got[r], want)
            assert np.all(got[r, m + 1:] == 0)
    cake.destroy()


def run_cascade_on(cake, w, indicators_dev, P):
    """Feeds indicators [L] of [H_kv][T] fp32 and preferences, runs every stage."""
    cake.begin(w.cu_seqlens)
    cake.set_preferences(torch.from_numpy(np.ascontiguousarray(P)).cuda())
    for l in range(w.n_layers):
        cake.set_indicators(l, indicators_dev[l])
        cake.allocate(l)
        cake.evict(l)


def test_cascade_and_compaction_bit_exact_on_oracle_indicators(case):
    w, qs, ks, vs, ref = case
    R, L, cu = len(w.seq_lens), w.n_layers, w.cu_seqlens
    T = w.total_tokens
    # the oracle's indicators rounded to fp32: both sides select from these values
    ind32 = []
    for l in range(L):
        full = np.zeros((w.n_kv_heads, T), dtype=np.float32)
        for r, N in enumerate(w.seq_lens):
            full[:, cu[r]:cu[r] + N - w.window] = ref[l][r]["indicator"].astype(np.float32)
        ind32.append(full)
    P = np.array([[ref[l][r]["P"] for l in range(L)] for r in range(R)], dtype=np.float64)
    cake = harness.cake_for(w)
    run_cascade_on(cake, w, [torch.from_numpy(x).cuda() for x in ind32], P)
    budgets = cake.get_budgets().cpu().numpy()
    k_out, v_out, off, pos = cake.compact(ks, vs)
    kb = harness.split_blocks(w, k_out, off)
    vb = harness.split_blocks(w, v_out, off)
    pb = harness.split_blocks(w, pos, off)
    assert cake.status() == 0
    for r, N in enumerate(w.seq_lens):
        n = N - w.window
        inds = [ind32[l][:, cu[r]:cu[r] + n].astype(np.float64) for l in range(L)]
        c = O.cascade(inds, P[r], total_budget=w.total_budget, window=w.window, seq_len=N)
        o = O.one_shot(inds, P[r], total_budget=w.total_budget, window=w.window, seq_len=N)
        assert np.array_equal(budgets[r], c.budgets)
        for l in range(L):
            got_pos = cake.get_positions(r, l, int(budgets[r, l])).cpu().numpy()
            for g in range(w.n_kv_heads):
                assert np.array_equal(got_pos[g], c.positions[l][g]), (r, l, g)
                assert np.array_equal(got_pos[g], o.positions[l][g])          # Theorem 2
                assert np.array_equal(pb[r][l][g].cpu().numpy(), c.positions[l][g])
            want_k, want_v = O.compact(ks[l][:, cu[r]:cu[r + 1]].cpu().view(torch.int16).numpy()
                                       if w.dtype == "bf16" else ks[l][:, cu[r]:cu[r + 1]].cpu().numpy(),
                                       vs[l][:, cu[r]:cu[r + 1]].cpu().view(torch.int16).numpy()
                                       if w.dtype == "bf16" else vs[l][:, cu[r]:cu[r + 1]].cpu().numpy(),
                                       c.positions[l])
            gk = kb[r][l].cpu()
            gv = vb[r][l].cpu()
            if w.dtype == "bf16":
                gk, gv = gk.view(torch.int16), gv.view(torch.int16)
            assert np.array_equal(gk.numpy(), want_k), (r, l)
            assert np.array_equal(gv.numpy(), want_v), (r, l)
    assert int(off[-1]) <= cake.packed_rows_bound()
    cake.destroy()


def test_end_to_end_own_indicators_differ_only_near_threshold(case):
    w, qs, ks, vs, ref = case
    R, L, cu = len(w.seq_lens), w.n_layers, w.cu_seqlens
    cake = harness.cake_for(w)
    k_out, v_out, off, pos = cake.run(qs, ks, vs, w.cu_seqlens)
    budgets = cake.get_budgets().cpu().numpy()
    pb = harness.split_blocks(w, pos, off)
    kb = harness.split_blocks(w, k_out, off)
    for r, N in enumerate(w.seq_lens):
        n = N - w.window
        inds = [ref[l][r]["indicator"] for l in range(L)]
        P = [ref[l][r]["P"] for l in range(L)]
        c = O.cascade(inds, P, total_budget=w.total_budget, window=w.window, seq_len=N)
        # budgets from the device's own preferences: reported, allowed to move by a few tokens
        assert np.abs(budgets[r] - c.budgets).max() <= 2, (budgets[r], c.budgets)
        for l in range(L):
            b = int(budgets[r, l]) - w.window
            for g in range(w.n_kv_heads):
                got = pb[r][l][g].cpu().numpy()
                assert len(got) == budgets[r, l] and np.all(np.diff(got) > 0)
                assert np.array_equal(got[b:], np.arange(n, N))
                # compacted rows are the source rows at the reported positions
                src = ks[l][g, cu[r] + torch.from_numpy(got).long().cuda()]
                assert torch.equal(kb[r][l][g], src)
                if b == 0 or b >= n:
                    continue
                want = O.topk_keep(inds[l][g], b)
                diff = np.setxor1d(got[:b], want)
                if diff.size:
                    thr = np.sort(inds[l][g])[::-1][b - 1]
                    rel = np.abs(inds[l][g][diff] - thr) / thr
                    assert rel.max() <= RTOL, (r, l, g, diff, rel.max())
    assert cake.status() == 0
    cake.destroy()


@pytest.mark.parametrize("mode,kind", [(1, "mean"), (2, "var"), (3, "mean*var")])
@pytest.mark.parametrize("name", ["tiny-fp32", "gqa-bf16"])
def test_indicator_modes_of_the_ablation(name, mode, kind):
    """The other combinations of window mean and variance (Section 5.3, Table "indicator_abl"),
    on the fp32 SIMT path and the bf16 tensor-core path."""
    w = SMALL_CASES[name]()
    qs, ks, vs = harness.device_inputs(w, layers=[0])
    cake = harness.cake_for(w, indicator_mode=mode)
    cake.begin(w.cu_seqlens)
    cake.score_layer(0, qs[0], ks[0])
    ind = cake.get_indicators(0).cpu().numpy()
    cu = w.cu_seqlens
    for r, N in enumerate(w.seq_lens):
        n = N - w.window
        ref = O.score_layer(to_np(qs[0][r]), to_np(ks[0][:, cu[r]:cu[r + 1]]), gamma=w.gamma,
                            pool_kernel=w.pool_kernel, tau1=w.tau1, tau2=w.tau2, indicator=kind)
        assert_close(ind[:, cu[r]:cu[r] + n], ref["indicator"], f"{kind} indicator, request {r}")
    assert cake.status() == 0
    cake.destroy()


@pytest.mark.parametrize("reserve", ["0", "40", "74"])
def test_score_is_the_same_for_any_share_of_the_sms(monkeypatch, reserve):
    """The score kernel's grid (and with it the plan: slices, segments, merge owners) follows
    the number of SMs left to the cascade kernels; the results must not."""
    monkeypatch.setenv("CAKE_RESERVED_SMS", reserve)
    w = SMALL_CASES["ragged"]()
    qs, ks, vs = harness.device_inputs(w)
    ref = oracle_scores(w, qs, ks)
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    cu = w.cu_seqlens
    for l in range(w.n_layers):
        cake.score_layer(l, qs[l], ks[l])
        ind = cake.get_indicators(l).cpu().numpy()
        for r, N in enumerate(w.seq_lens):
            n = N - w.window
            assert_close(ind[:, cu[r]:cu[r] + n], ref[l][r]["indicator"], f"layer {l} request {r}")
        cake.allocate(l)
        cake.evict(l)
    H, V, P = (x.cpu().numpy() for x in cake.get_preferences())
    for l in range(w.n_layers):
        for r in range(len(w.seq_lens)):
            assert_close(P[r, l], ref[l][r]["P"], f"P of layer {l} request {r}")
    assert cake.status() == 0
    cake.destroy()


# ------------------------------------------------ full size, as the benchmark launches it
def test_one_full_size_layer_of_the_128k_workload():
    """Layer 0 of the 128K Llama-3.1-8B-shaped workload at full length, in the launch
    configuration the benchmark times (same context geometry; only the layer count and the
    budget are scaled to one layer): every indicator and H, V, P against the oracle, then the
    selection on the device's own indicators, and the planted needles."""
    full = synth.workload(4)
    w = synth.scaled(full, n_layers=1, total_budget=full.total_budget // full.n_layers)
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    k_out, v_out, off, pos = cake.run(qs, ks, vs, w.cu_seqlens)
    assert cake.status() == 0
    N = w.seq_lens[0]
    n = N - w.window
    ref = O.score_layer(to_np(qs[0][0]), to_np(ks[0]), gamma=w.gamma, pool_kernel=w.pool_kernel,
                        tau1=w.tau1, tau2=w.tau2)
    ind = cake.get_indicators(0).cpu().numpy()
    assert_close(ind[:, :n], ref["indicator"], "indicator at 128K")
    H, V, P = (x.cpu().numpy() for x in cake.get_preferences())
    assert_close(H[0, 0], ref["H"], "H at 128K")
    assert_close(V[0, 0], ref["V"], "V at 128K")
    assert_close(P[0, 0], ref["P"], "P at 128K")
    b = int(cake.get_budgets().cpu().numpy()[0, 0]) - w.window
    assert b == w.total_budget - w.window
    got = harness.split_blocks(w, pos, off)[0][0].cpu().numpy()
    needles = np.array(synth.needle_positions(w, 0))
    for g in range(w.n_kv_heads):
        assert np.all(np.diff(got[g]) > 0) and np.array_equal(got[g][b:], np.arange(n, N))
        want = O.topk_keep(ref["indicator"][g], b)
        diff = np.setxor1d(got[g][:b], want)
        if diff.size:
            thr = np.sort(ref["indicator"][g])[::-1][b - 1]
            rel = np.abs(ref["indicator"][g][diff] - thr) / thr
            assert rel.max() <= RTOL, (g, diff.size, rel.max())
        if np.isin(needles, want).all():              # the oracle keeps every needle: so must we
            assert np.isin(needles, got[g][:b]).all(), g
        src = ks[0][g, torch.from_numpy(got[g]).long().cuda()]
        assert torch.equal(harness.split_blocks(w, k_out, off)[0][0][g], src)
    cake.destroy()


def test_four_full_size_layers_through_the_pipelined_cascade():
    """Four layers of the 128K workload, enqueued back to back as the benchmark does: while layer
    l+1 is scored, layer l is pooled, allocated and evicted on the library's own streams.  The
    preferences, the budgets and every retained set are checked against the oracle's cascade, and
    further batches in the same context must give the same bits."""
    full = synth.workload(4)
    L = 4
    w = synth.scaled(full, n_layers=L, total_budget=full.total_budget // full.n_layers * L)
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    k_out, v_out, off, pos = cake.run(qs, ks, vs, w.cu_seqlens)
    assert cake.status() == 0
    first = (pos.clone(), off.clone(), k_out.clone())
    N = w.seq_lens[0]
    n = N - w.window
    ref = [O.score_layer(to_np(qs[l][0]), to_np(ks[l]), gamma=w.gamma, pool_kernel=w.pool_kernel,
                         tau1=w.tau1, tau2=w.tau2) for l in range(L)]
    H, V, P = (x.cpu().numpy() for x in cake.get_preferences())
    for l in range(L):
        assert_close(H[0, l], ref[l]["H"], f"H of layer {l}")
        assert_close(V[0, l], ref[l]["V"], f"V of layer {l}")
        assert_close(P[0, l], ref[l]["P"], f"P of layer {l}")
    c = O.cascade([r["indicator"] for r in ref], [r["P"] for r in ref],
                  total_budget=w.total_budget, window=w.window, seq_len=N)
    budgets = cake.get_budgets().cpu().numpy()[0]
    assert budgets.sum() == w.total_budget
    assert np.abs(budgets - c.budgets).max() <= 2, (budgets, c.budgets)
    pb = harness.split_blocks(w, pos, off)
    kb = harness.split_blocks(w, k_out, off)
    for l in range(L):
        b = int(budgets[l]) - w.window
        for g in range(w.n_kv_heads):
            got = pb[0][l][g].cpu().numpy()
            assert len(got) == budgets[l] and np.all(np.diff(got) > 0)
            assert np.array_equal(got[b:], np.arange(n, N))
            want = O.topk_keep(ref[l]["indicator"][g], b)
            diff = np.setxor1d(got[:b], want)
            if diff.size:
                thr = np.sort(ref[l]["indicator"][g])[::-1][b - 1]
                rel = np.abs(ref[l]["indicator"][g][diff] - thr) / thr
                assert rel.max() <= RTOL, (l, g, diff.size, rel.max())
        g = l % w.n_kv_heads                               # one head's rows per layer, bit for bit
        src = ks[l][g, torch.from_numpy(pb[0][l][g].cpu().numpy()).long().cuda()]
        assert torch.equal(kb[0][l][g], src)
    for _ in range(6):                                     # the internal streams overlap differently each time
        k2, v2, off2, pos2 = cake.run(qs, ks, vs, w.cu_seqlens)
        assert cake.status() == 0
        assert torch.equal(off2, first[1]) and torch.equal(pos2, first[0]) and torch.equal(k2, first[2])
    cake.destroy()


# ---------------------------------------------------------------- edge cases
def small_w(**kw):
    base = synth.scaled(synth.workload(1), n_layers=2, seq_lens=(100,), total_budget=2 * 30)
    return synth.scaled(base, **kw)


def test_prompt_that_fits_is_kept_whole():
    w = small_w(seq_lens=(30, 17), total_budget=2 * 30)     # N <= B_total / L
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    k_out, v_out, off, pos = cake.run(qs, ks, vs, w.cu_seqlens)
    b = cake.get_budgets().cpu().numpy()
    assert np.array_equal(b, [[30, 30], [17, 17]])
    pb = harness.split_blocks(w, pos, off)
    kb = harness.split_blocks(w, k_out, off)
    for r, N in enumerate(w.seq_lens):
        for l in range(2):
            for g in range(w.n_kv_heads):
                assert np.array_equal(pb[r][l][g].cpu().numpy(), np.arange(N))
                assert torch.equal(kb[r][l][g], ks[l][g, w.cu_seqlens[r]:w.cu_seqlens[r + 1]])
    cake.destroy()


def test_window_plus_one_token_and_window_only_budget():
    w = small_w(seq_lens=(17, 40), total_budget=2 * 16)     # B' = 0: only the windows survive
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    k_out, v_out, off, pos = cake.run(qs, ks, vs, w.cu_seqlens)
    b = cake.get_budgets().cpu().numpy()
    assert np.array_equal(b, [[16, 16], [16, 16]])
    pb = harness.split_blocks(w, pos, off)
    for r, N in enumerate(w.seq_lens):
        for l in range(2):
            for g in range(w.n_kv_heads):
                assert np.array_equal(pb[r][l][g].cpu().numpy(), np.arange(N - 16, N))
    cake.destroy()


def test_budget_cap_at_non_window_tokens():
    # one preferred layer would get more than n tokens: capped, not redistributed
    w = small_w(seq_lens=(60,), total_budget=2 * 16 + 70)
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    P = np.array([[9.0, 1.0]])
    cake.set_preferences(torch.from_numpy(P).cuda())
    for m in range(2):
        cake.allocate(m)
        got = cake.get_budgets().cpu().numpy()[0, :m + 1]
        want = O.stage_budgets(P[0, :m + 1], w.total_budget, 2, 16, 60) + 16
        assert np.array_equal(got, want)
    assert got[0] == 60
    cake.destroy()


def test_zero_and_all_zero_preferences():
    w = small_w(n_layers=3, seq_lens=(200,), total_budget=3 * 16 + 50)
    cake = harness.cake_for(w)
    for P in ([[0.0, 2.0, 0.0]], [[0.0, 0.0, 0.0]], [[1e-300, 1e300, 1.0]], [[3.0, 3.0, 3.0]]):
        cake.begin(w.cu_seqlens)
        P = np.array(P)
        cake.set_preferences(torch.from_numpy(P).cuda())
        for m in range(3):
            cake.allocate(m)
            got = cake.get_budgets().cpu().numpy()[0, :m + 1]
            want = O.stage_budgets(P[0, :m + 1], w.total_budget, 3, 16, 200) + 16
            assert np.array_equal(got, want), (P, m, got, want)
        assert cake.status() == 0
    cake.begin(w.cu_seqlens)
    cake.set_preferences(torch.tensor([[1.0, float("nan"), 1.0]], dtype=torch.float64).cuda())
    cake.allocate(0)
    assert cake.status() == 0
    cake.allocate(1)
    assert cake.status() == -4                     # CAKE_ERR_NONFINITE, sticky
    cake.destroy()


def test_allocator_random_preferences_bit_exact():
    rng = np.random.default_rng(77)
    for trial in range(12):
        L = int(rng.integers(1, 33))
        Sw = 4
        B = L * Sw + int(rng.integers(0, 5000))
        N = int(rng.integers(Sw + 1, 4000))
        w = synth.scaled(synth.workload(1), n_layers=L, seq_lens=(N,), window=Sw, total_budget=B)
        cake = harness.cake_for(w)
        cake.begin(w.cu_seqlens)
        P = rng.random((1, L)) * 10.0 ** rng.integers(-6, 6, size=(1, L))
        if trial % 3 == 0:
            P = np.round(P * 4) / 4 + 0.25           # many exact ties between layers
        cake.set_preferences(torch.from_numpy(P).cuda())
        for m in range(L):
            cake.allocate(m)
            got = cake.get_budgets().cpu().numpy()[0, :m + 1]
            want = O.stage_budgets(P[0, :m + 1], B, L, Sw, N) + Sw
            assert np.array_equal(got, want), (trial, m, got, want)
        cake.destroy()


def test_selection_with_massive_ties_and_negative_values():
    w = small_w(n_layers=2, seq_lens=(5000,), total_budget=2 * 16 + 1500)
    rng = np.random.default_rng(5)
    T = w.total_tokens
    inds = [np.round(rng.normal(size=(w.n_kv_heads, T)) * 3).astype(np.float32) / 4 for _ in range(2)]
    inds[1][0, :] = 1.0                              # one head entirely tied
    P = np.array([[1.0, 2.5]])
    cake = harness.cake_for(w)
    run_cascade_on(cake, w, [torch.from_numpy(x).cuda() for x in inds], P)
    b = cake.get_budgets().cpu().numpy()
    c = O.cascade([x[:, :T - 16].astype(np.float64) for x in inds], P[0],
                  total_budget=w.total_budget, window=16, seq_len=T)
    assert np.array_equal(b[0], c.budgets)
    for l in range(2):
        got = cake.get_positions(0, l, int(b[0, l])).cpu().numpy()
        for g in range(w.n_kv_heads):
            assert np.array_equal(got[g], c.positions[l][g])
    cake.destroy()


def test_negative_zero_ties_with_positive_zero():
    """-0.0 and +0.0 are equal indicators: the lower position wins, as in the oracle."""
    w = small_w(n_layers=1, seq_lens=(400,), total_budget=16 + 100)
    T = w.total_tokens
    ind = np.full((w.n_kv_heads, T), -1.0, dtype=np.float32)
    ind[:, 0:300:2] = 0.0
    ind[:, 1:300:2] = -0.0
    ind[:, 350:360] = 1.0
    P = np.array([[1.0]])
    cake = harness.cake_for(w)
    run_cascade_on(cake, w, [torch.from_numpy(ind).cuda()], P)
    b = cake.get_budgets().cpu().numpy()
    c = O.cascade([ind[:, :T - 16].astype(np.float64)], P[0], total_budget=w.total_budget,
                  window=16, seq_len=T)
    got = cake.get_positions(0, 0, int(b[0, 0])).cpu().numpy()
    for g in range(w.n_kv_heads):
        assert np.array_equal(got[g], c.positions[0][g])
    cake.destroy()


def test_empty_batch_and_call_order_errors():
    w = small_w()
    cake = harness.cake_for(w)
    cake.begin([0])                                   # empty batch
    cake.score_layer(0, None, None)
    cake.allocate(0)
    cake.evict(0)
    qs, ks, vs = harness.device_inputs(w)
    cake.begin(w.cu_seqlens)
    with pytest.raises(CakeError) as e:
        cake.score_layer(1, qs[1], ks[1])             # layer 0 first
    assert e.value.code == CAKE_ERR_STATE
    with pytest.raises(CakeError) as e:
        cake.allocate(0)                              # no preference yet
    assert e.value.code == CAKE_ERR_STATE
    cake.score_layer(0, qs[0], ks[0])
    with pytest.raises(CakeError) as e:
        cake.evict(0)                                 # allocate first
    assert e.value.code == CAKE_ERR_STATE
    cake.allocate(0)
    cake.evict(0)
    with pytest.raises(CakeError) as e:
        cake.evict(0)
    assert e.value.code == CAKE_ERR_STATE
    with pytest.raises(CakeError) as e:
        cake.begin([0, 8])                            # shorter than the window
    assert e.value.code == CAKE_ERR_ARG
    with pytest.raises(CakeError) as e:
        cake.begin([0, 100, 300])                     # over capacity
    assert e.value.code == CAKE_ERR_CAPACITY
    cake.destroy()


def test_runs_are_bitwise_reproducible():
    w = SMALL_CASES["ragged"]()
    qs, ks, vs = harness.device_inputs(w)
    outs = []
    for _ in range(2):
        cake = harness.cake_for(w)
        k_out, v_out, off, pos = cake.run(qs, ks, vs, w.cu_seqlens)
        H, V, P = cake.get_preferences()
        outs.append((k_out.clone(), pos.clone(), off.clone(), P.clone()))
        cake.destroy()
    n = int(outs[0][2][-1])
    assert torch.equal(outs[0][2], outs[1][2])
    assert torch.equal(outs[0][0][:n], outs[1][0][:n])
    assert torch.equal(outs[0][1][:n], outs[1][1][:n])
    assert torch.equal(outs[0][3], outs[1][3])


def test_compaction_reads_values_from_pinned_host_memory():
    """V (and K) handed to the gather as page-locked host tensors give the same packed cache as
    device tensors: only the retained rows cross the bus."""
    w = SMALL_CASES["ragged"]()
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    k_dev, v_dev, off_dev, pos_dev = [t.clone() for t in cake.run(qs, ks, vs, w.cu_seqlens)]
    hv = [v.cpu().pin_memory() for v in vs]
    hk = [k.cpu().pin_memory() for k in ks]
    k_h, v_h, off_h, pos_h = cake.compact(hk, hv)
    n = int(off_dev[-1])
    assert n > 0 and torch.equal(off_dev, off_h)
    assert torch.equal(k_dev[:n], k_h[:n]) and torch.equal(v_dev[:n], v_h[:n])
    assert torch.equal(pos_dev[:n], pos_h[:n])
    with pytest.raises(ValueError):
        cake.compact(ks, [v.cpu() for v in vs])          # pageable host memory is refused
    cake.destroy()


def test_generator_is_bit_identical_on_cpu_and_gpu():
    w = SMALL_CASES["gqa-bf16"]()
    q0, k0, v0 = synth.layer_inputs(w, 1, "cpu")
    q1, k1, v1 = synth.layer_inputs(w, 1, "cuda")
    assert torch.equal(q0, q1.cpu()) and torch.equal(k0, k1.cpu()) and torch.equal(v0, v1.cpu())


def test_simt_and_tensor_core_paths_agree_on_bf16(monkeypatch):
    """bf16 inputs normally take the tcgen05 kernels; the SIMT kernels must give
    the same indicators and preferences (both within tolerance of the oracle)."""
    w = SMALL_CASES["gqa-bf16"]()
    qs, ks, vs = harness.device_inputs(w)
    ref = oracle_scores(w, qs, ks)
    res = {}
    for path in ("tc", "simt"):
        monkeypatch.setenv("CAKE_SCORE_PATH", path)
        cake = harness.cake_for(w)
        assert cake.uses_tensor_cores() == (path == "tc")
        cake.begin(w.cu_seqlens)
        inds = []
        for l in range(w.n_layers):
            cake.score_layer(l, qs[l], ks[l])
            inds.append(cake.get_indicators(l).cpu().numpy())
            cake.allocate(l)
            cake.evict(l)
        H, V, P = (x.cpu().numpy() for x in cake.get_preferences())
        assert cake.status() == 0
        res[path] = (inds, H, V, P)
        cake.destroy()
    n = w.seq_lens[0] - w.window
    for path in res:
        inds, H, V, P = res[path]
        for l in range(w.n_layers):
            assert_close(inds[l][:, :n], ref[l][0]["indicator"], f"{path} indicator l{l}")
            assert_close(H[0, l], ref[l][0]["H"], f"{path} H")
            assert_close(V[0, l], ref[l][0]["V"], f"{path} V")
    for l in range(w.n_layers):
        assert_close(res["tc"][0][l][:, :n], res["simt"][0][l][:, :n], "tc vs simt", rtol=1e-4)
