"""Textbook routines the oracle is pinned against (numpy / torch CPU, fp64)."""
import numpy as np
import torch


def softmax_attention(q, K, V, scale):
    """Eq. (att_score): softmax(q K^T * scale) V for q [G][d], K/V [n][d] -> (out [G][d], a [G][n])."""
    logits = (q @ K.T) * scale
    logits = logits - logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    a = p / p.sum(axis=1, keepdims=True)
    return a @ V, a


def sdpa_torch(q, K, V, scale):
    """The same through the library routine, fp64 on CPU."""
    tq = torch.from_numpy(np.ascontiguousarray(q))[None, :, None, :]          # [1, G, 1, d]
    tk = torch.from_numpy(np.ascontiguousarray(K))[None, None].expand(1, q.shape[0], -1, -1)
    tv = torch.from_numpy(np.ascontiguousarray(V))[None, None].expand(1, q.shape[0], -1, -1)
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=scale)
    return o[0, :, 0, :].numpy()


def causal_attention_matrix(Q, K, scale):
    """Rows tau of causal softmax attention for Q [T][d], K [T][d] -> A [T][T] (zero above the diagonal)."""
    T = K.shape[0]
    logits = (Q @ K.T) * scale
    mask = np.tril(np.ones((T, T), dtype=bool))
    logits = np.where(mask, logits, -np.inf)
    logits = logits - logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    return p / p.sum(axis=1, keepdims=True)


def heavy_hitter_stream(rng, n, d, G, frac=0.05):
    """Small random stream with a few keys aligned to the mean query (numpy, fp64)."""
    u = rng.normal(size=d)
    u /= np.linalg.norm(u)
    c = np.sqrt(4.0 * np.sqrt(d))
    q = rng.normal(size=(n, G, d)) + c * u
    k = rng.normal(size=(n, d))
    heavy = rng.random(n) < frac
    heavy[0] = True
    k[heavy] += c * u
    v = rng.normal(size=(n, d))
    return q, k, v
