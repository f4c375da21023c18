"""Glue between the synthetic workloads and the CUDA library (no method arithmetic)."""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch

from . import synth
from .binding import Cake


def cake_for(w: synth.Workload, **overrides) -> Cake:
    """A context sized for workload `w`."""
    kw = dict(n_layers=w.n_layers, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
              head_dim=w.head_dim, window=w.window, pool_kernel=w.pool_kernel, gamma=w.gamma,
              total_budget=w.total_budget, max_requests=max(1, len(w.seq_lens)),
              max_total_tokens=max(1, w.total_tokens), dtype=w.torch_dtype, tau1=w.tau1,
              tau2=w.tau2)
    kw.update(overrides)
    return Cake(**kw)


def device_inputs(w: synth.Workload, layers: Sequence[int] | None = None, device="cuda"
                  ) -> Tuple[List[torch.Tensor], List[torch.Tensor], List[torch.Tensor]]:
    """(Q_win, K, V) lists for the given layers, generated on `device`."""
    qs, ks, vs = [], [], []
    for l in (range(w.n_layers) if layers is None else layers):
        q, k, v = synth.layer_inputs(w, l, device)
        qs.append(q); ks.append(k); vs.append(v)
    return qs, ks, vs


def split_blocks(w: synth.Workload, packed: torch.Tensor, row_offsets: torch.Tensor
                 ) -> List[List[torch.Tensor]]:
    """Packed cache rows -> [req][layer] tensors of shape [H_kv][len][...]."""
    off = row_offsets.tolist()
    out = []
    for r in range(len(w.seq_lens)):
        per = []
        for l in range(w.n_layers):
            a, b = off[r * w.n_layers + l], off[r * w.n_layers + l + 1]
            blk = packed[a:b]
            per.append(blk.view(w.n_kv_heads, (b - a) // w.n_kv_heads, *packed.shape[1:]))
        out.append(per)
    return out
