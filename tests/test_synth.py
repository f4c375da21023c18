"""The seeded input generator: determinism, slice consistency, distribution,
and that the planted structure shows up in the oracle's result on the tiny
configuration (sinks and heavy hitters survive the cascade)."""
import numpy as np
import torch

from oracle import cake_oracle as O
from paper_2503_12491_b200 import synth


def test_gaussian_block_is_slice_consistent_and_roughly_normal():
    a = synth.gaussian_block(987654321, 0, 4096)
    b = synth.gaussian_block(987654321, 1000, 96)
    assert torch.equal(a[1000:1096], b)
    x = synth.gaussian_block(5, 0, 1 << 18).double()
    assert abs(x.mean().item()) < 0.01 and abs(x.std().item() - 1.0) < 0.01
    assert x.abs().max().item() < 6.0
    # exact in fp32: a multiple of 2^-16
    assert torch.equal((x * 65536).round(), x * 65536)
    assert not torch.equal(a, synth.gaussian_block(987654322, 0, 4096))


def test_workload_shapes_match_the_listed_configs():
    w1, w2, w3, w4, w5 = (synth.workload(i) for i in range(1, 6))
    assert (w1.n_layers, w1.n_q_heads, w1.n_kv_heads, w1.head_dim, w1.seq_lens, w1.window,
            w1.pool_kernel, w1.gamma, w1.total_budget, w1.dtype) == (4, 4, 4, 64, (512,), 16, 5, 1.0, 512, "fp32")
    assert (w2.n_q_heads, w2.n_kv_heads, w2.seq_lens, w2.total_budget) == (32, 32, (4096,), 32 * 1024)
    assert (w3.n_q_heads, w3.n_kv_heads, w3.seq_lens, w3.total_budget) == (32, 8, (32768,), 32 * 2048)
    assert (w4.seq_lens, w4.total_budget, w4.n_needles) == ((131072,), 32 * 4096, 16)
    assert len(w5.seq_lens) == 8 and all(8192 <= n <= 65536 for n in w5.seq_lens)
    assert w5.total_budget == 32 * 2048
    assert w5.seq_lens == synth.workload(5).seq_lens
    temps = [w4.temperature(l) for l in range(32)]
    assert min(temps) >= 0.5 and max(temps) <= 4.0 and len(set(temps)) == 32


def test_layer_inputs_are_deterministic_and_sliceable():
    w = synth.scaled(synth.workload(3), n_layers=2, seq_lens=(700, 300), total_budget=2 * 96)
    q, k, v = synth.layer_inputs(w, 1)
    q2, k2, v2 = synth.layer_inputs(w, 1, chunk_tokens=128)
    assert torch.equal(q, q2) and torch.equal(k, k2) and torch.equal(v, v2)
    assert k.shape == (8, 1000, 128) and k.dtype == torch.bfloat16 and q.shape == (2, 32, 32, 128)
    kk, vv = synth.kv_rows(w, 1, 1, 5, 17, 90)
    assert torch.equal(kk, k[5, 700 + 17:700 + 90]) and torch.equal(vv, v[5, 700 + 17:700 + 90])
    # sinks are boosted along the mean query: larger norm than ordinary keys
    assert k[0, :4].float().norm(dim=1).min() > k[0, 4:200].float().norm(dim=1).median()


def test_tiny_config_plants_survive_the_oracle_cascade():
    w = synth.workload(1)
    qs, ks = [], []
    for l in range(w.n_layers):
        q, k, _ = synth.layer_inputs(w, l)
        qs.append(q[0].numpy()); ks.append(k.numpy())
    out = O.run_request(qs, ks, gamma=w.gamma, pool_kernel=w.pool_kernel,
                        total_budget=w.total_budget)
    c = out["cascade"]
    assert c.budgets.sum() == w.total_budget
    H = [s["H"] for s in out["scored"]]
    assert H[0] > H[1] > H[2] > H[3]             # hotter layers are more dispersed
    for l in range(w.n_layers):
        for g in range(w.n_kv_heads):
            kept = set(c.positions[l][g].tolist())
            if c.budgets[l] - w.window >= 40:
                assert {0, 1, 2, 3} <= kept
                heavy = synth.heavy_positions(w, l, 0, g)
                assert len(kept & set(heavy)) >= 6
            else:                                # a starved layer keeps the strongest plants first
                assert min(kept) == 0
