"""cake_compact_int4 (INT4 keys per channel, values per token) against the oracle: codes, scales
and zeros bit for bit, on the rows and in the order cake_compact gives."""
import numpy as np
import pytest
import torch

from oracle import cake_oracle as O
from paper_2503_12491_b200 import synth, harness
from paper_2503_12491_b200.binding import CakeError, CAKE_ERR_ARG

pytestmark = pytest.mark.gpu


def to_f32(t):
    return t.detach().float().cpu().numpy()


@pytest.mark.parametrize("name,group", [("bf16-gqa", 32), ("bf16-gqa", 64), ("bf16-gqa", 128),
                                        ("fp32-mha-d64", 32), ("fp32-mha-d64", 64)])
def test_int4_compaction_bit_exact(name, group):
    if name == "bf16-gqa":
        w = synth.scaled(synth.workload(3), n_layers=3, n_q_heads=8, n_kv_heads=2, seq_lens=(1200, 333),
                         total_budget=3 * 150)
    else:
        w = synth.scaled(synth.workload(1), n_layers=2, seq_lens=(500, 77), total_budget=2 * 70)
    L, cu = w.n_layers, w.cu_seqlens
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    k_out, v_out, off, pos = cake.run(qs, ks, vs, cu)
    out = cake.compact_int4(ks, vs, group=group)
    assert cake.status() == 0
    n_rows = int(off[-1])
    assert torch.equal(out["row_offsets"], off) and torch.equal(out["positions"][:n_rows], pos[:n_rows])
    off_h = off.cpu().numpy()
    kg_h = out["kgroup_offsets"].cpu().numpy()
    budgets = cake.get_budgets().cpu().numpy()
    k_rows, v_rows = to_f32(k_out[:n_rows]), to_f32(v_out[:n_rows])     # the unquantised compaction
    k_codes, v_codes = out["k_codes"].cpu().numpy(), out["v_codes"].cpu().numpy()
    k_scale, k_zero = out["k_scale"].cpu().numpy(), out["k_zero"].cpu().numpy()
    v_scale, v_zero = out["v_scale"].cpu().numpy(), out["v_zero"].cpu().numpy()
    # values: per row
    q, s, z = O.quantize_values_per_token(v_rows, group)
    assert np.array_equal(v_codes[:n_rows], O.pack_nibbles(q))
    assert np.array_equal(v_scale[:n_rows], s) and np.array_equal(v_zero[:n_rows], z)
    # keys: per (request, layer, head), groups of consecutive packed rows
    groups_seen = 0
    for r in range(len(w.seq_lens)):
        for l in range(L):
            blk = r * L + l
            length = int(budgets[r, l])
            gpb = (length + group - 1) // group
            assert kg_h[blk + 1] - kg_h[blk] == w.n_kv_heads * gpb
            for g in range(w.n_kv_heads):
                a = off_h[blk] + g * length
                q, s, z = O.quantize_keys_per_channel(k_rows[a:a + length], group)
                assert np.array_equal(k_codes[a:a + length], O.pack_nibbles(q)), (r, l, g)
                ga = kg_h[blk] + g * gpb
                assert np.array_equal(k_scale[ga:ga + gpb], s) and np.array_equal(k_zero[ga:ga + gpb], z)
                groups_seen += gpb
    assert groups_seen == kg_h[-1]
    # reconstruction error of the values is at most half a step
    deq = np.repeat(v_zero[:n_rows], group, axis=1) + \
        np.stack([v_codes[:n_rows] & 15, v_codes[:n_rows] >> 4], axis=2).reshape(n_rows, -1) * \
        np.repeat(v_scale[:n_rows], group, axis=1)
    assert np.all(np.abs(deq - v_rows) <= 0.5 * np.repeat(v_scale[:n_rows], group, axis=1) * (1 + 1e-5) + 1e-7)
    cake.destroy()


def test_int4_compaction_rejects_bad_groups():
    w = synth.scaled(synth.workload(1), n_layers=1, seq_lens=(100,), total_budget=40)
    qs, ks, vs = harness.device_inputs(w)
    cake = harness.cake_for(w)
    cake.run(qs, ks, vs, w.cu_seqlens)
    for group in (16, 48, 128):                     # not offered, or wider than head_dim = 64
        with pytest.raises(CakeError) as e:
            cake.compact_int4(ks, vs, group=group)
        assert e.value.code == CAKE_ERR_ARG
    cake.destroy()
