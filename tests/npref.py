"""Independent numpy restatements used ONLY to pin the oracle (never by the CUDA path).

The rotary operator is written with complex numbers (pair (x0, x1) is the
complex number x0 + i x1, rotation by phi is multiplication by exp(i phi)),
attention with a library softmax: a different formulation from the oracle's
explicit real-valued loops, so a sign, index or transposition slip in either
shows up as a disagreement.
"""
from __future__ import annotations

import numpy as np
from scipy.special import logsumexp, softmax


def rope_np(x: np.ndarray, pos: np.ndarray, base: float = 10000.0) -> np.ndarray:
    """x [..., n, heads, d] float, pos [n, >=3] int -> rotated float64 (3D rotary, Sec. 3.1)."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    n_pairs = d // 2
    i = np.arange(n_pairs)
    axis = i % 3
    m = i // 3
    n_axis = np.array([(axis == a).sum() for a in range(3)])
    theta = base ** (-(m / n_axis[axis]))                       # [n_pairs]
    phi = np.asarray(pos)[:, :3][:, axis].astype(np.float64) * theta   # [n, n_pairs]
    z = x[..., 0::2] + 1j * x[..., 1::2]                          # [n, heads, n_pairs]
    z = z * np.exp(1j * phi)[:, None, :]
    out = np.empty_like(x)
    out[..., 0::2] = z.real
    out[..., 1::2] = z.imag
    return out


def logits_np(q, q_pos, k, k_pos, base=10000.0):
    """[Hq][n_q][n_k] scaled logits with GQA (query head h reads KV head h // G)."""
    rq, rk = rope_np(q, q_pos, base), rope_np(k, k_pos, base)
    hq, hkv, d = q.shape[1], k.shape[1], q.shape[2]
    g = hq // hkv
    rk_h = np.repeat(rk, g, axis=1)                               # [n_k][Hq][d]
    return np.einsum("ihd,jhd->hij", rq, rk_h) / np.sqrt(d)


def attend_np(q, q_pos, k, v, k_pos, base=10000.0, mask=None):
    """Returns (out [n_q][Hq][d], lse [n_q][Hq]); mask [n_q][n_k] True = visible."""
    lg = logits_np(q, q_pos, k, k_pos, base)
    if mask is not None:
        lg = np.where(mask[None], lg, -np.inf)
    p = softmax(lg, axis=-1)
    g = q.shape[1] // k.shape[1]
    v_h = np.repeat(np.asarray(v, dtype=np.float64), g, axis=1)   # [n_k][Hq][d]
    out = np.einsum("hij,jhd->ihd", p, v_h)
    return out, logsumexp(lg, axis=-1).T


def score_np(k, k_pos, q, q_pos, base=10000.0):
    """Mean scaled logit of each key over all queries and query heads."""
    return logits_np(q, q_pos, k, k_pos, base).mean(axis=(0, 1))


def attend_mass_np(q, q_pos, k, k_pos, base=10000.0):
    """Mean softmax probability each key receives over all (query, head) rows."""
    return softmax(logits_np(q, q_pos, k, k_pos, base), axis=-1).mean(axis=(0, 1))
