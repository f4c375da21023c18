"""Decode-time eviction with frozen budgets through the C-ABI against the oracle, in lockstep:
before every cake_decode_step the device's state of the layer (positions, scores, cache rows)
is read back, the oracle takes the same step from that state, and the two results are compared:
positions bit for bit, scores within 1e-3 relative, cache rows bit for bit.  Where the oracle's
two lowest scores lie within 1e-3 of each other the device may evict either (fp32 against
float64)."""
import numpy as np
import pytest
import torch

from oracle import cake_oracle as O
from paper_2503_12491_b200 import synth, harness
from paper_2503_12491_b200.binding import CAKE_POOL_AVG, CAKE_POOL_MAX, CakeError, CAKE_ERR_STATE

pytestmark = pytest.mark.gpu

RTOL = 1e-3
UPDATES = {0: "add", 1: "max", 2: "replace"}


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def read_heads(cake, w, r, l, length, k_cache, v_cache, off):
    """The device's decode state of block (r, l) as oracle DecodeHead objects."""
    pos, sc, sl = (x.cpu().numpy() for x in cake.decode_get_state(r, l, length))
    base = int(off[r * w.n_layers + l])
    cap = length + 1
    heads = []
    for g in range(w.n_kv_heads):
        rows = base + g * cap + torch.from_numpy(sl[g].astype(np.int64)).cuda()
        heads.append(O.DecodeHead(pos[g].astype(np.int64), sc[g][: length - w.window].astype(np.float64),
                                  to_np(k_cache[rows]), to_np(v_cache[rows])))
    return heads


def run_decode(w, steps, update_mode=0, pool_mode=CAKE_POOL_MAX):
    L, R, cu = w.n_layers, len(w.seq_lens), w.cu_seqlens
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w, pool_mode=pool_mode)
    k_out, v_out, poff, ppos = cake.run(qs, ks, vs, cu)
    budgets = cake.get_budgets().cpu().numpy()
    packed = harness.split_blocks(w, ppos, poff)
    k_cache, v_cache, off = cake.decode_begin(ks, vs, update_mode)
    assert cake.status() == 0
    off_h = off.cpu().numpy()
    # ---- the initial state: the compacted positions, the survivors' prefill indicators, the rows
    for r, N in enumerate(w.seq_lens):
        for l in range(L):
            length = int(budgets[r, l])
            heads = read_heads(cake, w, r, l, length, k_cache, v_cache, off_h)
            ref = O.score_layer(to_np(qs[l][r]), to_np(ks[l][:, cu[r]:cu[r + 1]]), gamma=w.gamma,
                                pool_kernel=w.pool_kernel, tau1=w.tau1, tau2=w.tau2,
                                pool_mode="max" if pool_mode == CAKE_POOL_MAX else "avg")
            for g in range(w.n_kv_heads):
                want_pos = packed[r][l][g].cpu().numpy()
                assert np.array_equal(heads[g].positions, want_pos)
                want = ref["indicator"][g][want_pos[: length - w.window]]
                assert np.allclose(heads[g].scores, want, rtol=RTOL, atol=1e-30)
                src = to_np(ks[l][g, cu[r] + torch.from_numpy(want_pos).long().cuda()])
                assert np.array_equal(heads[g].k, src)
    # ---- decode steps
    gen = torch.Generator().manual_seed(w.seed + 17)
    near_ties = 0
    for t in range(steps):
        for l in range(L):
            q_new = (torch.randn(R, w.n_q_heads, w.head_dim, generator=gen) * 1.5).to(w.torch_dtype).cuda()
            k_new = torch.randn(R, w.n_kv_heads, w.head_dim, generator=gen).to(w.torch_dtype).cuda()
            v_new = torch.randn(R, w.n_kv_heads, w.head_dim, generator=gen).to(w.torch_dtype).cuda()
            before = [read_heads(cake, w, r, l, int(budgets[r, l]), k_cache, v_cache, off_h) for r in range(R)]
            cake.decode_step(l, q_new, k_new, v_new, k_cache, v_cache)
            for r, N in enumerate(w.seq_lens):
                length = int(budgets[r, l])
                after = read_heads(cake, w, r, l, length, k_cache, v_cache, off_h)
                for g in range(w.n_kv_heads):
                    G = w.group
                    want, ev = O.decode_step_head(
                        before[r][g], to_np(q_new[r, g * G:(g + 1) * G]), to_np(k_new[r, g]), to_np(v_new[r, g]),
                        N + t, window=w.window, budget=length - w.window, pool_kernel=w.pool_kernel,
                        pool_mode="max" if pool_mode == CAKE_POOL_MAX else "avg", update=UPDATES[update_mode])
                    got = after[g]
                    assert len(got.positions) == length and np.all(np.diff(got.positions) > 0)
                    assert got.positions[-1] == N + t
                    if not np.array_equal(got.positions, want.positions):
                        # the device evicted another entry: only allowed at a near tie of the two
                        # lowest scores (recomputed by the oracle with nothing evicted)
                        full, _ = O.decode_step_head(
                            before[r][g], to_np(q_new[r, g * G:(g + 1) * G]), to_np(k_new[r, g]),
                            to_np(v_new[r, g]), N + t, window=w.window, budget=length, pool_kernel=w.pool_kernel,
                            pool_mode="max" if pool_mode == CAKE_POOL_MAX else "avg", update=UPDATES[update_mode])
                        gone_dev = np.setdiff1d(full.positions, got.positions)
                        assert len(gone_dev) == 1 and len(ev) == 1
                        s_dev = full.scores[np.searchsorted(full.positions, gone_dev[0])]
                        s_orc = full.scores[np.searchsorted(full.positions, ev[0])]
                        assert abs(s_dev - s_orc) <= RTOL * abs(s_orc), (t, l, r, g, s_dev, s_orc)
                        near_ties += 1
                        continue
                    assert np.allclose(got.scores, want.scores, rtol=RTOL, atol=1e-12), (t, l, r, g)
                    assert np.array_equal(got.k, want.k) and np.array_equal(got.v, want.v)
    assert cake.status() == 0
    cake.destroy()
    return near_ties


def test_decode_sixty_four_steps_bf16_gqa():
    w = synth.scaled(synth.workload(3), n_layers=2, n_q_heads=8, n_kv_heads=2, seq_lens=(900, 333),
                     total_budget=2 * 120)
    ties = run_decode(w, steps=64)
    assert ties <= 4


def test_decode_fp32_mha_with_average_pooling():
    w = synth.scaled(synth.workload(1), n_layers=2, seq_lens=(300, 150), total_budget=2 * 60)
    run_decode(w, steps=40, pool_mode=CAKE_POOL_AVG)


@pytest.mark.parametrize("mode", [1, 2])
def test_decode_other_update_readings(mode):
    w = synth.scaled(synth.workload(3), n_layers=1, n_q_heads=4, n_kv_heads=1, seq_lens=(500,),
                     total_budget=100)
    run_decode(w, steps=24, update_mode=mode)


@pytest.mark.parametrize("cluster", ["1", "0"])
def test_decode_large_heads(monkeypatch, cluster):
    """Heads of 512 slots or more are spread over a thread-block cluster; with that form switched
    off a head beyond the 5688 slots that G = 8 leaves in shared memory works in the context's
    global work area.  Both must match the oracle like the one-CTA form does."""
    monkeypatch.setenv("CAKE_DECODE_CLUSTER", cluster)
    w = synth.scaled(synth.workload(3), n_layers=1, n_q_heads=8, n_kv_heads=1, seq_lens=(7000, 400),
                     total_budget=6500, window=16)
    run_decode(w, steps=3)


def test_decode_cluster_form_over_many_steps():
    w = synth.scaled(synth.workload(3), n_layers=2, n_q_heads=8, n_kv_heads=2, seq_lens=(2500, 700),
                     total_budget=2 * 900)
    ties = run_decode(w, steps=24)
    assert ties <= 4


def test_decode_requires_a_finished_prefill():
    w = synth.scaled(synth.workload(1), n_layers=2, seq_lens=(100,), total_budget=2 * 30)
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    cake.score_layer(0, qs[0], ks[0]); cake.allocate(0); cake.evict(0)
    with pytest.raises(CakeError) as e:
        cake.decode_begin(ks, vs)
    assert e.value.code == CAKE_ERR_STATE
    cake.destroy()
