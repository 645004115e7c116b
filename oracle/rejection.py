"""Rejection-sampling acceptance (App. G) -- plain CPU restatement, test infrastructure only.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this module; the
product never does.

The rule, per verification stage (App. G, "Acceptance Rule in Rejection-Sampling"): the block
tokens S_1..S_n were drawn from the proposing exit's distributions p_k; the verifying exit gives
q_k at the same positions.  For k = 1..n in order: draw u_k ~ U(0,1); keep S_k if
u_k < min(1, q_k(S_k) / p_k(S_k)); at the first failure drop S_k and everything after it and draw a
replacement from the residual distribution max(0, q_k - p_k) / sum(max(0, q_k - p_k)).  If every
token is kept and the verifier computed one more row, the next token is drawn from that row's q.
Applied at L_i with (p, q) = (p_{L_d}, p_{L_i}) and at L_f with (p, q) = (p_{L_i}, p_{L_f}) (App. G,
"Lossless Guarantee under Rejection Sampling").

Random numbers are inputs (`u_accept`, `u_sample`), so the CUDA path can be compared draw by draw.
Probabilities are formed in fp32 -- the precision of the kernels -- because they decide integers.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np


def softmax_f32(logits: np.ndarray, temperature: float = 1.0) -> np.ndarray:
    """softmax(logits / temperature) over the last axis, fp32; -inf logits get probability 0."""
    z = np.asarray(logits, dtype=np.float32) * np.float32(1.0 / temperature)
    m = np.max(z, axis=-1, keepdims=True)
    e = np.exp(z - m, dtype=np.float32)
    return e / np.sum(e, axis=-1, keepdims=True, dtype=np.float32)


def sample_inverse_cdf(weights: np.ndarray, u: float) -> int:
    """Index v with  sum(weights[:v]) <= u * sum(weights) < sum(weights[:v+1])  (weights >= 0, not all 0):
    inversion sampling in vocabulary order.  Entries of weight 0 are never returned."""
    w = np.asarray(weights, dtype=np.float64)
    c = np.cumsum(w)
    target = float(u) * c[-1]
    v = int(np.searchsorted(c, target, side="right"))
    v = min(v, len(w) - 1)
    while w[v] == 0.0 and v > 0:      # u * total landed exactly on a boundary followed by empty entries
        v -= 1
    return v


def residual(p: Optional[np.ndarray], q: np.ndarray) -> np.ndarray:
    """max(0, q - p) (App. G); p None = no proposal at this row (bonus row): the residual is q itself."""
    if p is None:
        return np.asarray(q, dtype=np.float32)
    return np.maximum(np.float32(0.0), np.asarray(q, np.float32) - np.asarray(p, np.float32))


def rejection_verify(S: Sequence[int], p_rows: np.ndarray, q_rows: np.ndarray, u_accept: Sequence[float],
                     u_sample: float) -> Tuple[List[int], int]:
    """One verification stage.  p_rows [len(S)][V], q_rows [R][V] with R = len(S) or len(S) + 1 are
    probability rows.  Returns (result list, number of kept block tokens a): the kept tokens followed by
    the replacement (a < len(S)) or the bonus token (a == len(S) and R == len(S) + 1)."""
    n, R = len(S), q_rows.shape[0]
    assert R in (n, n + 1) and p_rows.shape[0] >= n
    a = 0
    while a < n:
        tok = int(S[a])
        pv, qv = np.float32(p_rows[a, tok]), np.float32(q_rows[a, tok])
        ratio = np.float32(1.0) if not pv > 0 else min(np.float32(1.0), qv / pv)
        if np.float32(u_accept[a]) < ratio:
            a += 1
        else:
            break
    out = [int(t) for t in S[:a]]
    if a < R:
        r = residual(p_rows[a] if a < n else None, q_rows[a])
        if not float(np.sum(r, dtype=np.float64)) > 0.0:   # p == q exactly: nothing left over, fall back to q
            r = np.asarray(q_rows[a], np.float32)
        out.append(sample_inverse_cdf(r, u_sample))
    return out, a
