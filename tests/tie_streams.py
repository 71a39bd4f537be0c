"""Constructed inputs in which the arg-max of Eq. (hatr) is an exact tie.

Sec. 3.4 sends an evicted token to the merged slot with the largest dot product; when two
slots give the same value the lowest slot takes it.  Random data never produces such a tie,
so these inputs plant them: pairs of merged slots (i < j) that are either bit-identical or
different keys with the same dot product against a chosen token, all in small integers so
every product and sum is exact in fp16, bf16, fp32 and fp64 alike, whatever the summation
order.  Input construction only: nothing of the method is computed here.
"""
from __future__ import annotations

import numpy as np


def planted_pairs(Br: int, d: int):
    """Slot pairs (i, j, kind): i from the front of the pool, j from the back, so that the two
    slots of a pair sit in different lanes, warps or row groups of whatever walks the pool."""
    n = min(4, Br // 2, d // 8)
    return [(m, Br - 1 - m, "identical" if m % 2 == 0 else "equal_dot") for m in range(n)]


def residual_fill_keys(rng, Br: int, d: int):
    """Keys of the first B_r evicted tokens (they take the free slots in order): small Gaussian
    fillers, with the planted pairs written over them.  Pair m lives on axis m."""
    K = np.round(rng.normal(size=(Br, d)) * 0.25 * 64) / 64          # exact in every dtype
    for m, (i, j, kind) in enumerate(planted_pairs(Br, d)):
        K[i] = 0.0
        K[j] = 0.0
        K[i, m] = K[j, m] = 8.0
        if kind == "equal_dot":                                      # different keys, same k_r . k_t
            K[i, d - 1 - 2 * m] = 3.0
            K[j, d - 2 - 2 * m] = -5.0
    return K


def tie_tokens(Br: int, d: int):
    """Keys that tie exactly between the two slots of each pair, and the slot each must go to.
    Round one: 8 e_m (dot 64 with both slots of pair m, at most a few units with any other
    slot).  Round two: 8 e_m + 4 e_x on an axis no slot uses, which ties again although slot i
    now has fusion count 2, and afterwards leaves the pair's keys different for good."""
    pairs = planted_pairs(Br, d)
    toks, want = [], []
    for rnd in range(2):
        for m, (i, j, _) in enumerate(pairs):
            k = np.zeros(d)
            k[m] = 8.0
            if rnd == 1:
                k[d // 2 + m] = 4.0
            toks.append(k)
            want.append(i)
    return np.array(toks).reshape(-1, d), want


def planted_prompt(rng, d: int, Bp: int, Bc: int, Br: int, n_more: int):
    """A prompt whose evicted stream (ascending position) is: B_r slot fillers with planted
    pairs, the tie tokens, then n_more ordinary tokens.  Returns K, V [T][d], the scores to
    supply (the evicted positions share the lowest value; the kept ones lie far above), the
    number of evicted positions and the merge targets the tie tokens must get."""
    fill = residual_fill_keys(rng, Br, d)
    ties, want = tie_tokens(Br, d)
    more = np.round(rng.normal(size=(n_more, d)) * 16) / 16
    keep = np.round(rng.normal(size=(Bc + Bp, d)) * 16) / 16
    K = np.concatenate([fill, ties, more, keep])
    T = K.shape[0]
    V = np.round(rng.normal(size=(T, d)) * 16) / 16
    n_ev = Br + len(want) + n_more
    scores = np.empty(T, np.float32)
    scores[:n_ev] = 0.25
    scores[n_ev:] = 1.0 + rng.random(T - n_ev).astype(np.float32)
    return K, V, scores, n_ev, want
