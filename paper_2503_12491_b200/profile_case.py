"""A reduced case of the eviction path, sized for profiler captures.

    python -m paper_2503_12491_b200.profile_case [--workload 4] [--layers 2] [--steps 1] [--lse]

Runs the first `--layers` layers of a benchmark workload (same shapes per layer,
budget scaled with the layer count) through begin / score / allocate / evict /
compact.  Every layer's K is still larger than the L2 cache at workloads 4 and 5,
so DRAM counters stay meaningful, while only a few GB are held on the device and
a capture that replays each kernel many times ends by itself.  With --lse the
window rows' log-sum-exps are computed beforehand (plain torch, as a fused attention
forward would hand them over) and passed to cake_score_layer, so the score kernel runs
its column pass only.  Prints the time of the last step; that figure is for orientation
only, never a benchmark value.

Two more measurements of the rows that follow the prefill path, each timed with CUDA events:
--int4 GROUP times cake_compact_int4 beside cake_compact on the evicted layers; --decode T
builds the decode cache and times T tokens of cake_decode_step over all layers (one launch per
layer and token) after one untimed token.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import harness, synth


def window_lse(w, q, k) -> torch.Tensor:
    """Natural-log sum-exp of every window row's scaled logits over its visible keys:
    the input a caller passes as `lse` ([n_req][H_q][S_w] fp32)."""
    cu = w.cu_seqlens
    out = torch.empty(len(w.seq_lens), w.n_q_heads, w.window, dtype=torch.float32, device=q.device)
    for r, N in enumerate(w.seq_lens):
        i = torch.arange(w.window, device=q.device)[:, None]
        j = torch.arange(N, device=q.device)[None, :]
        for g in range(w.n_kv_heads):
            qg = q[r][g * w.group:(g + 1) * w.group].float()
            s = torch.einsum("hid,jd->hij", qg, k[g, cu[r]:cu[r + 1]].float()) / (w.head_dim ** 0.5)
            s = s.masked_fill(j > (N - w.window) + i, float("-inf"))
            out[r, g * w.group:(g + 1) * w.group] = torch.logsumexp(s, dim=-1)
    return out


def _timed(fn, reps: int) -> float:
    """Mean milliseconds of `fn` over `reps` calls, CUDA events on the current stream."""
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def time_int4(cake, w, ks, vs, bufs, group: int) -> dict:
    """cake_compact_int4 against cake_compact on the same retained sets."""
    rows = int(bufs["row_offsets"][-1])
    esize = 4 if w.dtype == "fp32" else 2
    ms_bf = _timed(lambda: cake.compact(ks, vs, **bufs), 5)
    ms_q = _timed(lambda: cake.compact_int4(ks, vs, group), 5)   # includes the outputs' allocation
    read = 2 * rows * w.head_dim * esize
    return {"group": group, "rows": rows, "compact_ms": ms_bf, "compact_int4_ms": ms_q,
            "bytes_read": read, "compact_GBps": 2 * read / ms_bf * 1e-6,
            "int4_bytes_written": rows * w.head_dim + 2 * 4 * rows * (w.head_dim // group) +
            2 * 4 * (rows // group) * w.head_dim,
            "int4_read_GBps": read / ms_q * 1e-6}


def time_decode(cake, w, ks, vs, tokens: int) -> dict:
    """Decode-time eviction: `tokens` new tokens, every layer evicted back to its frozen budget."""
    L, R = w.n_layers, len(w.seq_lens)
    k_cache, v_cache, off = cake.decode_begin(ks, vs, 0)
    budgets = cake.get_budgets()
    gen = torch.Generator(device="cuda").manual_seed(w.seed + 99)
    q_new = (torch.randn(R, w.n_q_heads, w.head_dim, generator=gen, device="cuda") * 1.5).to(w.torch_dtype)
    k_new = torch.randn(R, w.n_kv_heads, w.head_dim, generator=gen, device="cuda").to(w.torch_dtype)
    v_new = torch.randn(R, w.n_kv_heads, w.head_dim, generator=gen, device="cuda").to(w.torch_dtype)

    def token():
        for l in range(L):
            cake.decode_step(l, q_new, k_new, v_new, k_cache, v_cache)

    ms = _timed(token, tokens)
    esize = 4 if w.dtype == "fp32" else 2
    slots = int(budgets.sum().item()) * w.n_kv_heads            # K rows read per token, all layers
    return {"tokens": tokens, "ms_per_token": ms, "us_per_layer_step": ms / L * 1e3,
            "k_bytes_per_token": slots * w.head_dim * esize,
            "k_GBps": slots * w.head_dim * esize / ms * 1e-6,
            "slots_per_head_min": int(budgets.min().item()), "slots_per_head_max": int(budgets.max().item())}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=4)
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--steps", type=int, default=1)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--lse", action="store_true", help="supply the window rows' log-sum-exps")
    ap.add_argument("--int4", type=int, default=0, metavar="GROUP",
                    help="also time the INT4 compaction with this group size (32, 64 or 128)")
    ap.add_argument("--decode", type=int, default=0, metavar="T",
                    help="also time T tokens of decode-time eviction over all layers")
    args = ap.parse_args()

    full = synth.workload(args.workload)
    L = max(1, min(args.layers, full.n_layers))
    w = synth.scaled(full, n_layers=L, total_budget=full.total_budget // full.n_layers * L)
    torch.cuda.set_device(0)
    qs, ks, vs = harness.device_inputs(w)
    lses = [window_lse(w, qs[l], ks[l]) for l in range(L)] if args.lse else None
    cake = harness.cake_for(w)
    cake.begin(w.cu_seqlens)
    rows = cake.packed_rows_bound()
    bufs = dict(k_out=torch.empty(rows, w.head_dim, dtype=w.torch_dtype, device="cuda"),
                v_out=torch.empty(rows, w.head_dim, dtype=w.torch_dtype, device="cuda"),
                row_offsets=torch.empty(len(w.seq_lens) * L + 1, dtype=torch.int64, device="cuda"),
                positions=torch.empty(rows, dtype=torch.int32, device="cuda"))
    ms = None
    for it in range(args.warmup + args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if lses is None:
            cake.run(qs, ks, vs, w.cu_seqlens, **bufs)
        else:
            cake.begin(w.cu_seqlens)
            for l in range(L):
                cake.score_layer(l, qs[l], ks[l], lse=lses[l])
                cake.allocate(l)
                cake.evict(l)
            cake.compact(ks, vs, **bufs)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
    out = {"workload": w.name, "layers": L, "tokens": w.total_tokens, "last_step_ms": ms,
           "retained_rows": int(bufs["row_offsets"][-1])}
    if args.int4:
        out["int4"] = time_int4(cake, w, ks, vs, bufs, args.int4)
    if args.decode:
        out["decode"] = time_decode(cake, w, ks, vs, args.decode)
    status = cake.status()
    out["device_status"] = status
    print(json.dumps(out))
    cake.destroy()
    if status != 0:
        raise SystemExit(1)


if __name__ == "__main__":
    main()
