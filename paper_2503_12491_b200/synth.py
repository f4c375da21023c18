"""Seeded synthetic Q/K/V with planted attention structure.

This module serves both the CUDA path and the CPU oracle's tests.  It holds no
arithmetic of the eviction method itself: it only manufactures inputs.  Every
element is a pure function of (seed, tensor, request, layer, head, token, dim),
computed with 64-bit integer hashing plus a handful of IEEE fp32 multiply/add
operations, so a CPU tensor and a CUDA tensor of the same workload are
bit-identical and any slice can be regenerated without materialising the rest.

The workloads stand in for the long-context benchmarks the paper evaluates on
(Section 5.1: LongBench / NeedleBench prompts through Llama-2-7B,
Mistral-7B and Llama-3.1-8B); only the shapes and the qualitative structure
the paper describes are reproduced -- a few "sink" and heavy-hitter keys
(Section 3), per-layer differences in dispersion and shift (Figure 2), a band
of recent keys, and planted "needle" keys.

Element recipe
--------------
counter = stream_key + 3*(token*d + dim) + {0,1,2}; three splitmix64-style
finalisers give twelve 16-bit lanes whose sum S is Irwin-Hall distributed;
x = (S - 393210) / 65536 is ~N(0,1), |x| < 6, and exact in fp32.

    Q_win = t_l * x                       (temperature on the query side)
    K     = x + beta_j * u_{l,g}          (planted boosts)
    V     = x

each rounded once to the workload dtype.  u_{l,g} points along the mean window
query of KV-head g's group and is scaled so that beta = 1 raises a key's mean
window logit by one logit standard deviation t_l.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import torch

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB

TENSOR_Q, TENSOR_K, TENSOR_V = 1, 2, 3
_TAG_TEMP, _TAG_HEAVY, _TAG_NEEDLE, _TAG_LEN = 11, 12, 13, 14


def _s64(x: int) -> int:
    """Python int (mod 2**64) -> the signed value an int64 tensor would hold."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_py(z: int) -> int:
    """splitmix64 finaliser on a Python int."""
    z = (z + _GOLDEN) & _M64
    z = ((z ^ (z >> 30)) * _MUL1) & _M64
    z = ((z ^ (z >> 27)) * _MUL2) & _M64
    return z ^ (z >> 31)


def hash_py(*words: int) -> int:
    """Order-sensitive 64-bit hash of a tuple of integers (host side)."""
    h = 0x243F6A8885A308D3
    for w in words:
        h = _mix_py(h ^ (int(w) & _M64))
    return h


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    """Logical shift right on int64 storage."""
    return (z >> k) & ((1 << (64 - k)) - 1)


def _mix_t(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on an int64 tensor (wrapping arithmetic)."""
    z = z + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_MUL1)
    z = (z ^ _lsr(z, 27)) * _s64(_MUL2)
    return z ^ _lsr(z, 31)


def gaussian_block(stream_key: int, first: int, count: int,
                   device: torch.device | str = "cpu") -> torch.Tensor:
    """fp32 tensor of `count` pseudo-normal values for flat element indices
    first .. first+count-1 of the stream `stream_key`."""
    idx = torch.arange(first, first + count, dtype=torch.int64, device=device)
    base = idx * 3 + _s64(stream_key)
    total = torch.zeros(count, dtype=torch.int64, device=device)
    for j in range(3):
        h = _mix_t(base + j)
        total += (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)
    return (total - 393210).to(torch.float32) * (1.0 / 65536.0)


@dataclass(frozen=True)
class Workload:
    """Shape, hyper-parameters and planting recipe of one benchmark config."""
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq_lens: Tuple[int, ...]            # one prompt length per request
    window: int                          # S_w
    pool_kernel: int
    gamma: float
    total_budget: int                    # B_total per request
    dtype: str                           # "fp32" | "bf16"
    seed: int
    tau1: float = 1.0
    tau2: float = 1.0
    temperatures: Tuple[float, ...] = ()  # empty => seeded log-uniform in [0.5, 4]
    n_sinks: int = 4
    n_heavy: int = 0                     # >0: that many keys; 0: 1 % of keys
    band: int = 0                        # keys just before the window boosted +1
    n_needles: int = 0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def total_tokens(self) -> int:
        return sum(self.seq_lens)

    @property
    def cu_seqlens(self) -> List[int]:
        out = [0]
        for n in self.seq_lens:
            out.append(out[-1] + n)
        return out

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    def temperature(self, layer: int) -> float:
        if self.temperatures:
            return float(self.temperatures[layer % len(self.temperatures)])
        u = (hash_py(self.seed, _TAG_TEMP, layer) >> 11) / float(1 << 53)
        return math.exp(math.log(0.5) + u * (math.log(4.0) - math.log(0.5)))


_BASE_SEED = 250312491


def _ragged_lengths(seed: int, count: int, lo: int, hi: int) -> Tuple[int, ...]:
    return tuple(lo + hash_py(seed, _TAG_LEN, r) % (hi - lo + 1) for r in range(count))


def workload(index: int) -> Workload:
    """The five benchmark configurations (1-based, as they are listed)."""
    if index == 1:
        return Workload("tiny-fp32", 4, 4, 4, 64, (512,), 16, 5, 1.0, 4 * 128, "fp32",
                        _BASE_SEED + 1, temperatures=(0.5, 1.0, 2.0, 4.0), n_heavy=8)
    if index == 2:
        return Workload("llama2-7b-4k", 32, 32, 32, 128, (4096,), 32, 7, 200.0, 32 * 1024,
                        "bf16", _BASE_SEED + 2, band=256)
    if index == 3:
        return Workload("mistral-7b-gqa-32k", 32, 32, 8, 128, (32768,), 32, 7, 200.0,
                        32 * 2048, "bf16", _BASE_SEED + 3, band=256)
    if index == 4:
        return Workload("llama31-8b-gqa-128k", 32, 32, 8, 128, (131072,), 32, 7, 200.0,
                        32 * 4096, "bf16", _BASE_SEED + 4, band=256, n_needles=16)
    if index == 5:
        lens = _ragged_lengths(_BASE_SEED + 5, 8, 8192, 65536)
        return Workload("llama31-8b-gqa-ragged", 32, 32, 8, 128, lens, 32, 7, 200.0,
                        32 * 2048, "bf16", _BASE_SEED + 5, band=256, n_needles=16)
    raise ValueError(f"no workload {index}")


def scaled(w: Workload, **changes) -> Workload:
    """A copy of `w` with some fields replaced (reduced-size test cases)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(changes)
    return Workload(**d)


def _stream(w: Workload, tensor: int, req: int, layer: int, head: int) -> int:
    return hash_py(w.seed, tensor, req, layer, head)


def window_queries_req(w: Workload, layer: int, req: int, device="cpu") -> torch.Tensor:
    """Q_win of one (layer, request): [H_q][S_w][d] in the workload dtype."""
    t = torch.tensor(w.temperature(layer), dtype=torch.float32, device=device)
    per_head = w.window * w.head_dim
    out = torch.empty(w.n_q_heads, w.window, w.head_dim, dtype=w.torch_dtype, device=device)
    for h in range(w.n_q_heads):
        x = gaussian_block(_stream(w, TENSOR_Q, req, layer, h), 0, per_head, device)
        out[h] = (x * t).to(w.torch_dtype).view(w.window, w.head_dim)
    return out


def window_queries(w: Workload, layer: int, device="cpu") -> torch.Tensor:
    """Q_win of one layer: [n_req][H_q][S_w][d] in the workload dtype."""
    return torch.stack([window_queries_req(w, layer, r, device)
                        for r in range(len(w.seq_lens))])


def boost_direction(w: Workload, layer: int, req: int) -> torch.Tensor:
    """u_{l,g}: [H_kv][d] fp32 (always computed on the host in float64)."""
    q = window_queries_req(w, layer, req).to(torch.float64)
    q = q.view(w.n_kv_heads, w.group * w.window, w.head_dim)
    m = q.mean(dim=1)                                            # [H_kv][d]
    t = w.temperature(layer)
    scale = t * math.sqrt(w.head_dim) / (m * m).sum(dim=1, keepdim=True).clamp_min(1e-300)
    return (m * scale).to(torch.float32)


def heavy_positions(w: Workload, layer: int, req: int, head: int) -> List[int]:
    """Explicit heavy-hitter positions (only when the workload plants a fixed count)."""
    n = w.seq_lens[req] - w.window
    out: List[int] = []
    c = 0
    while len(out) < min(w.n_heavy, max(n - w.n_sinks, 0)):
        p = w.n_sinks + hash_py(w.seed, _TAG_HEAVY, req, layer, head, c) % (n - w.n_sinks)
        c += 1
        if p not in out:
            out.append(p)
    return sorted(out)


def needle_positions(w: Workload, req: int) -> List[int]:
    """Needle token positions of a request (shared by all layers and heads)."""
    n = w.seq_lens[req] - w.window
    lo, hi = w.n_sinks, n - w.band
    out: List[int] = []
    c = 0
    while len(out) < w.n_needles and hi > lo + w.n_needles:
        p = lo + hash_py(w.seed, _TAG_NEEDLE, req, c) % (hi - lo)
        c += 1
        if p not in out:
            out.append(p)
    return sorted(out)


def boost_profile(w: Workload, layer: int, req: int, head: int,
                  lo: int, hi: int, device="cpu") -> torch.Tensor:
    """beta_j for tokens lo..hi-1 of one (request, layer, KV head): fp32 [hi-lo].
    Categories overlap by taking the largest boost."""
    N = w.seq_lens[req]
    n = N - w.window
    j = torch.arange(lo, hi, dtype=torch.int64, device=device)
    beta = torch.zeros(hi - lo, dtype=torch.float32, device=device)
    if w.band > 0:
        beta = torch.where((j >= n - w.band) & (j < n), torch.ones_like(beta), beta)
    if w.n_heavy > 0:
        for p in heavy_positions(w, layer, req, head):
            if lo <= p < hi:
                beta[p - lo] = max(float(beta[p - lo]), 2.0)
    else:
        hk = hash_py(w.seed, _TAG_HEAVY, req, layer, head)
        hv = _lsr(_mix_t(j + _s64(hk)), 1) % 100
        beta = torch.where((hv == 0) & (j >= w.n_sinks) & (j < n),
                           torch.full_like(beta, 2.0).maximum(beta), beta)
    beta = torch.where(j < w.n_sinks, torch.full_like(beta, 3.0), beta)
    for p in needle_positions(w, req):
        if lo <= p < hi:
            beta[p - lo] = 4.0
    return beta


def kv_rows(w: Workload, layer: int, req: int, head: int, lo: int, hi: int,
            device="cpu", u: torch.Tensor | None = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """K and V rows lo..hi-1 of one (request, layer, KV head): [hi-lo][d] each."""
    d = w.head_dim
    if u is None:
        u = boost_direction(w, layer, req)
    uh = u[head].to(device)
    xk = gaussian_block(_stream(w, TENSOR_K, req, layer, head), lo * d, (hi - lo) * d, device)
    beta = boost_profile(w, layer, req, head, lo, hi, device)
    k = xk.view(hi - lo, d) + beta[:, None] * uh[None, :]
    xv = gaussian_block(_stream(w, TENSOR_V, req, layer, head), lo * d, (hi - lo) * d, device)
    return k.to(w.torch_dtype), xv.view(hi - lo, d).to(w.torch_dtype)


def layer_inputs(w: Workload, layer: int, device="cpu",
                 chunk_tokens: int = 1 << 16) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """(Q_win, K, V) of one layer.  K and V are packed varlen
    [H_kv][sum N_r][d]; request r owns rows cu[r]..cu[r+1]-1 of every head."""
    q = window_queries(w, layer, device)
    T = w.total_tokens
    k = torch.empty(w.n_kv_heads, T, w.head_dim, dtype=w.torch_dtype, device=device)
    v = torch.empty_like(k)
    cu = w.cu_seqlens
    for r, N in enumerate(w.seq_lens):
        u = boost_direction(w, layer, r)
        for g in range(w.n_kv_heads):
            for lo in range(0, N, chunk_tokens):
                hi = min(N, lo + chunk_tokens)
                kk, vv = kv_rows(w, layer, r, g, lo, hi, device, u)
                k[g, cu[r] + lo:cu[r] + hi] = kk
                v[g, cu[r] + lo:cu[r] + hi] = vv
    return q, k, v


def planted_summary(w: Workload, layer: int, req: int, head: int) -> Dict[str, List[int]]:
    """Positions of the planted keys of one (request, layer, head), for reports."""
    N = w.seq_lens[req]
    beta = boost_profile(w, layer, req, head, 0, N)
    return {
        "sinks": list(range(min(w.n_sinks, N))),
        "heavy": torch.nonzero(beta == 2.0).flatten().tolist(),
        "needles": needle_positions(w, req),
    }
