"""CPU oracle for the attention-rollout analysis.  TEST INFRASTRUCTURE ONLY.

Plain numpy in float64, written from the definitions in Section 2.1 of the paper ("Analysis of audio-visual
token importance via attention rollout", Eq. 2 and Eq. 3).  Nothing here is shared with the CUDA library.

    A^l            head-mean of the layer's attention weights, one n x n row-stochastic matrix per layer
    Eq. 2          A~^l = alpha A^l + (1 - alpha) I
    Eq. 3          R^l = A~^l A~^(l-1) ... A~^1          (the newest layer multiplies from the left)

Readings where the paper is silent: the attention weights are the model's own (softmax of scale * q.k over
the keys a row may see, causal by index, query head h reading KV head h // G); alpha is a parameter; the
importance of input token j is the mean over rows of column j of R (Section 2.1 after Eq. 3: the influence of
each input-layer token on all tokens); the threshold keeps the tokens whose importance reaches it, and the
positional rule the paper derives from it is "keep everything before the last such token".
"""
from __future__ import annotations

import numpy as np


def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def attention_map(q_bits, k_bits, scale: float, causal: bool = True) -> np.ndarray:
    """A^l of one layer: q [n, Hq, d], k [n, Hkv, d] as bf16 bit patterns -> [n, n] float64.

    Row i is token i's attention distribution over the tokens it may see (j <= i when causal), averaged over
    the Hq query heads."""
    q, k = _bf16_to_f64(q_bits), _bf16_to_f64(k_bits)
    n, hq, d = q.shape
    hkv = k.shape[1]
    assert k.shape[0] == n and k.shape[2] == d and hq % hkv == 0
    group = hq // hkv
    out = np.zeros((n, n), dtype=np.float64)
    for h in range(hq):
        z = scale * (q[:, h, :] @ k[:, h // group, :].T)                     # [n, n] logits of head h
        if causal:
            z = np.where(np.arange(n)[None, :] <= np.arange(n)[:, None], z, -np.inf)
        z = z - z.max(axis=1, keepdims=True)
        p = np.exp(z)
        out += p / p.sum(axis=1, keepdims=True)
    return out / hq


def with_residual(a: np.ndarray, alpha: float) -> np.ndarray:
    """Eq. 2."""
    a = np.asarray(a, dtype=np.float64)
    return alpha * a + (1.0 - alpha) * np.eye(a.shape[0])


def rollout(maps, alpha: float) -> np.ndarray:
    """Eq. 3 over the given per-layer attention matrices, first layer first."""
    r = None
    for a in maps:
        a_tilde = with_residual(a, alpha)
        r = a_tilde if r is None else a_tilde @ r
    return r


def importance(r: np.ndarray) -> np.ndarray:
    """Influence of each input token on the tokens of the current layer: the column means of R."""
    return np.asarray(r, dtype=np.float64).mean(axis=0)


def threshold_rule(imp: np.ndarray, threshold: float, protect=None):
    """Tokens whose importance reaches the threshold (or that are protected) are kept.  Returns the keep mask
    (uint8) and the cut position: one past the last unprotected token that reaches the threshold (0 if none)."""
    imp = np.asarray(imp)
    reach = imp >= threshold
    keep = reach.copy()
    if protect is not None:
        keep |= np.asarray(protect).astype(bool)
    idx = np.nonzero(reach if protect is None else reach & ~np.asarray(protect).astype(bool))[0]
    return keep.astype(np.uint8), int(idx[-1]) + 1 if len(idx) else 0
