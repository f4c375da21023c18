"""CPU oracle for CAKE's prefill-time eviction path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 NumPy statement of what the path computes, written from
the paper's definitions.  It shares no code with the CUDA library and must never
be imported by the product: only the tests, the smoke check and the benchmark's
CPU-baseline leg call it.  Nothing here is blocked, fused or reordered beyond
what the definitions say: the S_w x N window attention matrix of every head is
materialised in full.

Readings taken where the paper is silent or ambiguous (each is also a
parameter so the alternative can be exercised):
  * softmax scale is 1/sqrt(head_dim)                       (Section 2, Eq. 2)
  * the observed slice A[-S_w:, :-S_w] is not renormalised  (Eq. 6, Listing 1)
  * natural logarithm in the dispersion                     (Eq. 4)
  * population variance (ddof = 0)                          (Eq. 5, Eq. 11)
  * heads -> layer: mean over query heads of H_h and of V_h, then Eq. 6
                                                             (Appendix "More
                                                             Implementation Details")
  * grouped-query models: the indicator is built from the attention averaged
    over the query heads that share a KV head; H_h, V_h stay per query head
  * pooling: max, stride 1, same length, window clipped at both ends;
    alternative: average with zero padding                  (Section 4.3)
  * the layer budget includes the observation window, which is always kept:
    every layer owns S_w slots, the remaining B' = B_total - L*S_w
    "selectable" slots are split by Eq. 7 / Eq. 9
  * integer budgets: Webster / Sainte-Lague highest averages on B'
    (priorities P_l/(s+1/2); ties: lower layer, then lower s) -- sums exactly
    and never grows a layer's budget when a layer is added (Proposition 1)
  * budgets are capped at the number of non-window tokens, the excess is not
    redistributed (Listing 1); a prompt with N <= floor(B_total/L) is kept whole
  * TopK order: indicator descending, token position ascending   (Eq. 12)
  * stored indicators of survivors are kept as they are (Section 4.2)
  * compacted rows in ascending token position, window last      (Eq. 12)
  * decode-time eviction: see the section of that name below

Pins: tests/test_oracle_pins.py checks every function below against closed
forms, invariants the paper states (Proposition 1, Theorem 2), special cases
(gamma = 0, kernel 1, single layer) and brute force on tiny inputs.  What no
pin can decide from the paper's text -- max versus average pooling, ddof,
whether the budget counts the window, how the decode step's "update_score"
combines old and new values, and the rounding rule of the 4-bit compaction --
is "parity unpinned" beyond those readings.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# window attention                                            (Section 2, Eq. 2)
# --------------------------------------------------------------------------
def window_logits(q_win: np.ndarray, k: np.ndarray) -> np.ndarray:
    """s[h,i,j] = q_{h,i} . k_{g(h),j} / sqrt(d) for the last S_w queries against
    all N keys; key j is masked (-inf) for window row i when j > (N - S_w) + i.

    q_win: [H_q][S_w][d], k: [H_kv][N][d]  ->  [H_q][S_w][N]
    Query head h reads KV head h // (H_q/H_kv).                       (Eq. 2)
    """
    q = np.asarray(q_win, dtype=F64)
    kk = np.asarray(k, dtype=F64)
    Hq, Sw, d = q.shape
    Hkv, N, _ = kk.shape
    G = Hq // Hkv
    n = N - Sw
    s = np.empty((Hq, Sw, N), dtype=F64)
    for h in range(Hq):
        s[h] = q[h] @ kk[h // G].T / np.sqrt(F64(d))
    i = np.arange(Sw)[:, None]
    j = np.arange(N)[None, :]
    s[:, j > n + i] = -np.inf
    return s


def softmax_rows(s: np.ndarray) -> np.ndarray:
    """Row softmax with the row maximum subtracted.                    (Eq. 2)"""
    m = s.max(axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / e.sum(axis=-1, keepdims=True)


def observed_attention(q_win: np.ndarray, k: np.ndarray) -> np.ndarray:
    """A[-S_w:, :-S_w] per query head, rows not renormalised.   (Eq. 6, Listing 1)"""
    Sw = q_win.shape[1]
    A = softmax_rows(window_logits(q_win, k))
    return A[:, :, : A.shape[2] - Sw]


# --------------------------------------------------------------------------
# layer preference                                       (Section 3, Eq. 4-6)
# --------------------------------------------------------------------------
def dispersion(a_obs: np.ndarray) -> np.ndarray:
    """H(A) = -sum_i A[i,:] . log A[i,:]  per head (0 log 0 = 0).       (Eq. 4)"""
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(a_obs > 0, a_obs * np.log(a_obs), 0.0)
    return -t.sum(axis=(-2, -1))


def shift(a_obs: np.ndarray, ddof: int = 0) -> np.ndarray:
    """V(A) = sum_j Var(A[:,j])  per head.                              (Eq. 5)"""
    if a_obs.shape[-1] == 0:
        return np.zeros(a_obs.shape[:-2], dtype=F64)
    return a_obs.var(axis=-2, ddof=ddof).sum(axis=-1)


def layer_preference(a_obs: np.ndarray, tau1: float, tau2: float,
                     ddof: int = 0) -> Tuple[float, float, float]:
    """(H_l, V_l, P_l): head means of Eq. 4 and Eq. 5, then
    P = H^(1/tau1) * V^(1/tau2).                                        (Eq. 6)"""
    H = F64(dispersion(a_obs).mean()) if a_obs.size else F64(0.0)
    V = F64(shift(a_obs, ddof).mean()) if a_obs.size else F64(0.0)
    P = np.power(H, F64(1.0) / F64(tau1)) * np.power(V, F64(1.0) / F64(tau2))
    return float(H), float(V), float(P)


# --------------------------------------------------------------------------
# eviction indicator                                      (Section 4.3, Eq. 11)
# --------------------------------------------------------------------------
INDICATOR_KINDS = ("mean+var", "mean", "var", "mean*var", "sum")


def indicator_raw(a_obs: np.ndarray, n_kv_heads: int, gamma: float,
                  ddof: int = 0, kind: str = "mean+var") -> np.ndarray:
    """I[g,n] = Mean_i(Abar[g,:,n]) + gamma * Var_i(Abar[g,:,n]) for the
    non-window tokens, Abar = attention averaged over the group's query heads.
    [H_q][S_w][n] -> [H_kv][n]                                        (Eq. 11)
    `kind` selects the other combinations of the paper's indicator ablation
    (Section 5.3, Table "indicator_abl"): the mean alone, the variance alone,
    their product."""
    assert kind in INDICATOR_KINDS
    Hq, Sw, n = a_obs.shape
    G = Hq // n_kv_heads
    abar = a_obs.reshape(n_kv_heads, G, Sw, n).mean(axis=1)
    if n == 0:
        return np.zeros((n_kv_heads, 0), dtype=F64)
    mean = abar.mean(axis=1)
    var = abar.var(axis=1, ddof=ddof)
    if kind == "mean":
        return mean
    if kind == "var":
        return var
    if kind == "mean*var":
        return mean * var
    if kind == "sum":                       # SnapKV's window sum (Section 5.3, compatibility study)
        return abar.sum(axis=1)
    return mean + F64(gamma) * var


def pool1d(x: np.ndarray, kernel: int, mode: str = "max") -> np.ndarray:
    """Stride-1, same-length pooling along the last axis over [0, n) only.
    "max": window clipped at the ends; "avg": zero padding, divisor `kernel`.
                                                                (Section 4.3)"""
    assert kernel >= 1 and kernel % 2 == 1
    n = x.shape[-1]
    r = kernel // 2
    out = np.empty_like(x, dtype=F64)
    for j in range(n):
        lo, hi = max(0, j - r), min(n, j + r + 1)
        if mode == "max":
            out[..., j] = x[..., lo:hi].max(axis=-1)
        else:
            out[..., j] = x[..., lo:hi].sum(axis=-1) / F64(kernel)
    return out


def score_layer(q_win: np.ndarray, k: np.ndarray, *, gamma: float, pool_kernel: int,
                tau1: float = 1.0, tau2: float = 1.0, ddof: int = 0,
                pool_mode: str = "max", indicator: str = "mean+var") -> Dict[str, object]:
    """Everything one layer contributes before the cascade: pooled indicator
    [H_kv][n] and (H_l, V_l, P_l).                    (Algorithm 1, lines 4-5)"""
    a_obs = observed_attention(q_win, k)
    H, V, P = layer_preference(a_obs, tau1, tau2, ddof)
    raw = indicator_raw(a_obs, k.shape[0], gamma, ddof, indicator)
    return {"indicator": pool1d(raw, pool_kernel, pool_mode), "indicator_raw": raw,
            "H": H, "V": V, "P": P}


# --------------------------------------------------------------------------
# budgets                                        (Section 4.1-4.2, Eq. 7, Eq. 9)
# --------------------------------------------------------------------------
def webster(prefs: Sequence[float], seats: int) -> np.ndarray:
    """Integer split of `seats` in proportion to `prefs` by highest averages
    with divisors s + 1/2: the `seats` largest of P_l/(s+1/2) win; ties go to
    the lower layer, then the lower s.  All-zero preferences are treated as
    all-equal; a zero preference among positive ones gets nothing.
    Integerises B_l = P_l / sum(P) * B.                           (Eq. 7, Eq. 9)"""
    P = np.asarray(prefs, dtype=F64)
    if not np.all(np.isfinite(P)) or np.any(P < 0):
        raise ValueError("preferences must be finite and non-negative")
    L = P.shape[0]
    out = np.zeros(L, dtype=np.int64)
    if seats <= 0 or L == 0:
        return out
    if not np.any(P > 0):
        P = np.ones(L, dtype=F64)
    s = np.arange(seats, dtype=F64)
    pri = P[:, None] / (s[None, :] + F64(0.5))                  # [L][seats]
    layer = np.repeat(np.arange(L), seats)
    step = np.tile(np.arange(seats), L)
    flat = pri.ravel()
    live = flat > 0
    order = np.lexsort((step[live], layer[live], -flat[live]))   # value desc, layer asc, s asc
    won = layer[live][order[:seats]]
    np.add.at(out, won, 1)
    return out


ALLOC_MODES = ("preference", "uniform", "pyramid")


def allocation_weights(prefs: Sequence[float], n_layers: int, mode: str = "preference",
                       slope: float = 0.0) -> np.ndarray:
    """What the budget split of the layers seen so far is proportional to: the
    preferences (Eq. 7 / Eq. 9), or one of the fixed patterns the paper's allocation
    ablation compares with (Section 5.3): the same weight for every layer, or weights
    falling linearly with the layer index, w_l = 1 + slope*(L-1-2l)/(L-1) (an arithmetic
    progression with mean 1 over all L layers; slope in [0, 1])."""
    assert mode in ALLOC_MODES
    m1 = len(prefs)
    if mode == "preference":
        return np.asarray(prefs, dtype=F64)
    if mode == "uniform" or n_layers <= 1:
        return np.ones(m1, dtype=F64)
    l = np.arange(m1, dtype=F64)
    return F64(1.0) + F64(slope) * (F64(n_layers - 1) - 2.0 * l) / F64(n_layers - 1)


def cumulative_attention(q_all: np.ndarray, k: np.ndarray) -> np.ndarray:
    """H2O's indicator: the attention every key has received from ALL prompt queries
    (causal softmax rows summed over the queries), averaged over the group's query heads.
    q_all: [H_q][N][d], k: [H_kv][N][d] -> [H_kv][N].  It needs the whole prefill
    attention and is not computed by the window-score path; a caller that has it hands it
    to the cascade in place of Eq. 11's indicator (Section 5.3, compatibility study)."""
    q = np.asarray(q_all, dtype=F64)
    kk = np.asarray(k, dtype=F64)
    Hq, N, d = q.shape
    Hkv = kk.shape[0]
    G = Hq // Hkv
    out = np.zeros((Hkv, N), dtype=F64)
    mask = np.triu(np.ones((N, N), dtype=bool), 1)
    for h in range(Hq):
        s = q[h] @ kk[h // G].T / np.sqrt(F64(d))
        s[mask] = -np.inf
        out[h // G] += softmax_rows(s).sum(axis=0) / G
    return out


def stage_budgets(prefs_seen: Sequence[float], total_budget: int, n_layers: int,
                  window: int, seq_len: int) -> np.ndarray:
    """Selectable (non-window) budgets b_l^{(m)} of the layers seen so far.
    B' = B_total - L*S_w is split over the seen layers (Eq. 9), each capped at
    n = N - S_w (Listing 1, `min(budget, seq_len - window)`); a prompt with
    N <= floor(B_total / L) keeps everything."""
    n = seq_len - window
    m1 = len(prefs_seen)
    if total_budget < n_layers * window:
        raise ValueError("total budget smaller than the layers' windows")
    if seq_len <= total_budget // n_layers:
        return np.full(m1, n, dtype=np.int64)
    b = webster(prefs_seen, total_budget - n_layers * window)
    return np.minimum(b, n)


# --------------------------------------------------------------------------
# EVICT                                     (Section 4.2, Section 4.3, Eq. 12)
# --------------------------------------------------------------------------
def topk_keep(values: np.ndarray, k: int) -> np.ndarray:
    """Indices (ascending) of the k entries that come first in the order
    (value descending, index ascending).                               (Eq. 12)"""
    n = values.shape[0]
    k = max(0, min(int(k), n))
    order = np.lexsort((np.arange(n), -np.asarray(values, dtype=F64)))
    return np.sort(order[:k])


@dataclass
class LayerState:
    """What the cascade stores for one layer: per KV head the surviving
    non-window positions (ascending) and their pooled indicators."""
    positions: List[np.ndarray]
    values: List[np.ndarray]


@dataclass
class CascadeResult:
    budgets: np.ndarray                       # [L] retained length per layer incl. window
    positions: List[List[np.ndarray]]         # [L][H_kv] ascending token positions incl. window
    stage_budgets: List[np.ndarray] = field(default_factory=list)   # selectable budgets per stage
    stage_positions: List[List[List[np.ndarray]]] = field(default_factory=list)


def cascade(indicators: Sequence[np.ndarray], prefs: Sequence[float], *, total_budget: int,
            window: int, seq_len: int, keep_history: bool = False) -> CascadeResult:
    """Algorithm 1.  indicators[l]: pooled [H_kv][n]; prefs[l]: P_l.  After layer
    m arrives the budgets of layers 0..m are recomputed (Eq. 9) and every one of
    them is shrunk to its budget by TopK on its *stored* indicators; survivors
    keep their indicator values.  The window tokens are always retained."""
    L = len(indicators)
    n = seq_len - window
    win = np.arange(n, seq_len, dtype=np.int64)
    states: List[LayerState] = []
    res = CascadeResult(np.zeros(L, dtype=np.int64), [])
    b = np.zeros(0, dtype=np.int64)
    for m in range(L):
        ind = np.asarray(indicators[m], dtype=F64)
        states.append(LayerState([np.arange(n, dtype=np.int64) for _ in range(ind.shape[0])],
                                 [ind[g].copy() for g in range(ind.shape[0])]))
        b = stage_budgets(prefs[: m + 1], total_budget, L, window, seq_len)
        for l in range(m + 1):
            st = states[l]
            for g in range(len(st.positions)):
                keep = topk_keep(st.values[g], b[l])
                st.positions[g] = st.positions[g][keep]
                st.values[g] = st.values[g][keep]
        if keep_history:
            res.stage_budgets.append(b.copy())
            res.stage_positions.append([[p.copy() for p in st.positions] for st in states])
    res.budgets = np.array([int(b[l]) + window for l in range(L)], dtype=np.int64)
    res.positions = [[np.concatenate([p, win]) for p in st.positions] for st in states]
    return res


def one_shot(indicators: Sequence[np.ndarray], prefs: Sequence[float], *, total_budget: int,
             window: int, seq_len: int) -> CascadeResult:
    """The non-cascading strategy of Section 4.1: all preferences known, one
    budget split (Eq. 7), one TopK per layer and head (Eq. 12).  Theorem 2 says
    `cascade` must return the same sets."""
    L = len(indicators)
    n = seq_len - window
    win = np.arange(n, seq_len, dtype=np.int64)
    b = stage_budgets(prefs, total_budget, L, window, seq_len)
    pos = []
    for l in range(L):
        ind = np.asarray(indicators[l], dtype=F64)
        pos.append([np.concatenate([topk_keep(ind[g], b[l]), win]) for g in range(ind.shape[0])])
    return CascadeResult(np.array([int(x) + window for x in b], dtype=np.int64), pos)


def compact(k: np.ndarray, v: np.ndarray, positions: Sequence[np.ndarray]
            ) -> Tuple[np.ndarray, np.ndarray]:
    """K_hat = K[D,:], V_hat = V[D,:] per KV head; [H_kv][N][d] -> [H_kv][len][d].
                                                                       (Eq. 12)"""
    kh = np.stack([k[g][np.asarray(positions[g])] for g in range(k.shape[0])])
    vh = np.stack([v[g][np.asarray(positions[g])] for g in range(v.shape[0])])
    return kh, vh


# --------------------------------------------------------------------------
# quantised compaction       (Appendix "Comparison and Compatibility with
#                             Quantization Methods": KIVI-INT4 with CAKE)
# --------------------------------------------------------------------------
# Asymmetric 4-bit codes of the compacted rows, keys per channel and values per
# token.  The code is an integer decided by floating point, so the arithmetic is
# fixed: IEEE float32, zero = min, scale = (max - min)/15 (1 if max = min),
# code = clip(rint((x - zero)/scale), 0, 15) with round-half-to-even.
F32 = np.float32


def int4_codes(x: np.ndarray, axis: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Codes (uint8, 0..15), scale and zero (float32, `axis` kept with length 1) of one
    group spanning `axis`."""
    x = np.asarray(x, dtype=F32)
    zero = x.min(axis=axis, keepdims=True)
    span = (x.max(axis=axis, keepdims=True) - zero).astype(F32)
    scale = np.where(span > 0, (span / F32(15.0)).astype(F32), F32(1.0)).astype(F32)
    q = np.rint(((x - zero).astype(F32) / scale).astype(F32))
    return np.clip(q, 0, 15).astype(np.uint8), scale, zero


def quantize_values_per_token(v_rows: np.ndarray, group: int):
    """v_rows [rows][d] -> codes [rows][d], scale, zero [rows][d/group]: groups of
    `group` consecutive channels of a row."""
    rows, d = v_rows.shape
    x = np.asarray(v_rows, dtype=F32).reshape(rows, d // group, group)
    q, s, z = int4_codes(x, axis=2)
    return q.reshape(rows, d), s[..., 0], z[..., 0]


def quantize_keys_per_channel(k_rows: np.ndarray, group: int):
    """k_rows [len][d] (one head's compacted rows) -> codes [len][d], scale, zero
    [ceil(len/group)][d]: per channel, groups of `group` consecutive rows (the last
    group may be shorter)."""
    n, d = k_rows.shape
    codes = np.zeros((n, d), dtype=np.uint8)
    scales, zeros = [], []
    for t0 in range(0, n, group):
        q, s, z = int4_codes(np.asarray(k_rows[t0:t0 + group], dtype=F32), axis=0)
        codes[t0:t0 + group] = q
        scales.append(s[0])
        zeros.append(z[0])
    return codes, np.array(scales, dtype=F32).reshape(-1, d), np.array(zeros, dtype=F32).reshape(-1, d)


def pack_nibbles(codes: np.ndarray) -> np.ndarray:
    """[rows][d] codes -> [rows][d/2] bytes, the even channel in the low nibble."""
    return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)


# --------------------------------------------------------------------------
# decode-time eviction        (Section 5.1 "Implementation Details"; Appendix
#                              "More Implementation Details"; Listing 1, the
#                              branches taken when not prefilling)
# --------------------------------------------------------------------------
# After the prefill every layer's budget is frozen at its final allocation.  Per
# generated token and layer the new token's K/V is appended, the new token's
# attention over the cached keys is pooled and "updates" the stored scores, and
# the layer is evicted back to its frozen budget; the S_w most recent tokens are
# always kept.  Readings (the listing leaves them open; "parity unpinned"):
#   * observed attention of the single new query: softmax over ALL cached keys
#     (the new one included), columns of the S_w most recent tokens dropped, not
#     renormalised -- the one-row case of Eq. 6's slice;
#   * grouped-query models: mean over the group's query heads, as in the prefill;
#   * pooling runs over the cache in ascending token position (the order the
#     listing keeps the compressed cache in), same mode and kernel as the prefill;
#   * `update_score`: the pooled value is ADDED to the stored score ("add",
#     default); the token that has just left the window has no stored score and
#     starts from its pooled value.  "max" and "replace" are the alternatives;
#   * eviction: TopK of Eq. 12 with the frozen budget on the stored scores
#     (score descending, position ascending), per KV head.
DECODE_UPDATES = ("add", "max", "replace")


@dataclass
class DecodeHead:
    """Decode-time cache of one (layer, KV head): entries in ascending token
    position; the last `window` entries are the recent window and carry no score."""
    positions: np.ndarray        # [c] int64
    scores: np.ndarray           # [c - window] float64, stored eviction scores
    k: np.ndarray                # [c][d]
    v: np.ndarray                # [c][d]


def decode_attention(q_new: np.ndarray, k_cache: np.ndarray) -> np.ndarray:
    """softmax(q k^T / sqrt(d)) of one new query per head over all cached keys.
    q_new: [G][d] (the query heads of one KV head), k_cache: [c][d] -> [G][c]   (Eq. 2)"""
    q = np.asarray(q_new, dtype=F64)
    k = np.asarray(k_cache, dtype=F64)
    s = q @ k.T / np.sqrt(F64(q.shape[-1]))
    return softmax_rows(s)


def decode_step_head(h: DecodeHead, q_new: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
                     position: int, *, window: int, budget: int, pool_kernel: int,
                     pool_mode: str = "max", update: str = "add") -> Tuple[DecodeHead, np.ndarray]:
    """One decode step of one (layer, KV head).  Returns the new state and the
    positions that were evicted (normally one)."""
    assert update in DECODE_UPDATES
    pos = np.concatenate([h.positions, [position]]).astype(np.int64)
    k = np.concatenate([h.k, np.asarray(k_new)[None, :]], axis=0)
    v = np.concatenate([h.v, np.asarray(v_new)[None, :]], axis=0)
    c = pos.shape[0]
    n_obs = c - window                       # entries outside the recent window
    if n_obs <= 0:
        return DecodeHead(pos, np.zeros(0, dtype=F64), k, v), np.zeros(0, dtype=np.int64)
    a = decode_attention(q_new, k)           # [G][c]
    abar = a[:, :n_obs].mean(axis=0)         # observed slice, group mean
    pooled = pool1d(abar[None, :], pool_kernel, pool_mode)[0]
    old = h.scores.shape[0]                  # entries that already carry a score
    scores = np.empty(n_obs, dtype=F64)
    if update == "add":
        scores[:old] = h.scores + pooled[:old]
    elif update == "max":
        scores[:old] = np.maximum(h.scores, pooled[:old])
    else:
        scores[:old] = pooled[:old]
    scores[old:] = pooled[old:]              # tokens that have just left the window
    keep = topk_keep(scores, budget)         # indices into the non-window entries, ascending
    evicted = np.setdiff1d(np.arange(n_obs), keep)
    sel = np.concatenate([keep, np.arange(n_obs, c)])
    return DecodeHead(pos[sel], scores[keep], k[sel], v[sel]), pos[evicted]


def decode_init(k: np.ndarray, v: np.ndarray, positions: Sequence[np.ndarray],
                indicator: np.ndarray, window: int) -> List[DecodeHead]:
    """Decode-time state of one layer from the prefill's result: retained positions
    per KV head (ascending, window last) and the stored indicators of the survivors."""
    out = []
    for g in range(k.shape[0]):
        p = np.asarray(positions[g], dtype=np.int64)
        nw = p[: p.shape[0] - window]
        out.append(DecodeHead(p, np.asarray(indicator[g], dtype=F64)[nw].copy(), k[g][p], v[g][p]))
    return out


# --------------------------------------------------------------------------
# whole request
# --------------------------------------------------------------------------
def run_request(q_layers: Sequence[np.ndarray], k_layers: Sequence[np.ndarray], *,
                gamma: float, pool_kernel: int, total_budget: int, tau1: float = 1.0,
                tau2: float = 1.0, ddof: int = 0, pool_mode: str = "max",
                keep_history: bool = False) -> Dict[str, object]:
    """Score every layer, then run Algorithm 1.  q_layers[l]: [H_q][S_w][d],
    k_layers[l]: [H_kv][N][d]."""
    Sw = q_layers[0].shape[1]
    N = k_layers[0].shape[1]
    scored = [score_layer(q, k, gamma=gamma, pool_kernel=pool_kernel, tau1=tau1, tau2=tau2,
                          ddof=ddof, pool_mode=pool_mode) for q, k in zip(q_layers, k_layers)]
    res = cascade([s["indicator"] for s in scored], [s["P"] for s in scored],
                  total_budget=total_budget, window=Sw, seq_len=N, keep_history=keep_history)
    return {"scored": scored, "cascade": res}
