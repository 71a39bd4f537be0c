"""Attention-output error of the compressed cache against full attention, residual merging
versus pure eviction (the numerical error analysis of the paper's Sec. 4.3, on synthetic data).

Everything runs in the library's kernels: the reference is the same decode kernel on a cache
whose budget holds the whole context (nothing is ever evicted, so its output is plain softmax
attention); the two candidates are caches of `ratio * prompt_len` slots per head, one with
the recommended residual share and alpha = 1, one with B_r = 0.  All three see the same prompt
(one-shot compression after prefill) and the same decode inputs; the error of a step is
||o - o_full|| / ||o_full|| per query head, averaged over heads and steps.

    python -m paper_2503_10714_b200.error_analysis [--prompt 4096 --steps 128 ...]

The paper does not state its data or protocol, so only the ordering (merging below eviction at
every ratio) is comparable with its figure, not the values.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

import workloads as wl
from . import binding as zb


class _Cache:
    def __init__(self, w, bp, bc, br, alpha, lam=0.98, similarity=0):
        self.w = w
        full = lambda x: np.full((w.n_layers, w.n_kv_heads), int(x), dtype=np.int32)
        self.cfg = zb.make_config(w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype,
                                  full(bp), full(bc), full(br), lam=lam, alpha=alpha,
                                  similarity=similarity)
        self.buf = torch.empty(zb.zsm_cache_bytes(self.cfg), dtype=torch.uint8, device="cuda")
        self.h = zb.zsm_cache_create(self.cfg, self.buf)
        self.out = torch.empty(w.n_layers, w.batch, w.n_q_heads, w.head_dim, dtype=w.torch_dtype,
                               device="cuda")

    def prefill(self, layer, K, V, Qw, ws):
        zb.zsm_prefill_compress(self.h, layer, K, V, Qw, None, K.shape[2], Qw.shape[2], ws)

    def step(self, q, k, v):
        zb.zsm_decode_step(self.h, -1, q, k, v, self.out)
        return self.out.float()

    def close(self):
        zb.zsm_cache_free(self.h)


def run(ratios=(0.5, 0.2, 0.1, 0.05), prompt_len=4096, steps=128, n_layers=2, batch=2, heads=8,
        head_dim=128, dtype="f16", window=32, seed=41, tail_ratio=0.5, dense_ratio=0.02,
        alpha=1.0, lam=0.98, similarity=0):
    """Mean relative output error per ratio for merging and for eviction.  Returns a dict
    {ratio: {"merge": e, "evict": e, "reduction": 1 - merge/evict, "slots": B, "B_r": r}}."""
    w = wl.Workload("error_analysis", n_layers, batch, heads, heads, head_dim, dtype, prompt_len,
                    steps, window, None, seed)
    dev = "cuda"
    u = wl.directions(w, dev)
    ref = _Cache(w, 0, prompt_len + steps, 0, 1.0)
    cands = {}
    for r in ratios:
        B = max(4, int(round(r * prompt_len)))
        bp, bc, br = zb.zsm_split_budget(B, tail_ratio, dense_ratio)
        bp0, bc0, _ = zb.zsm_split_budget(B, tail_ratio, 0.0)
        cands[r] = (B, br, _Cache(w, bp, bc, br, alpha, lam, similarity),
                    _Cache(w, bp0, bc0, 0, 1.0, lam))
    caches = [ref] + [c for v in cands.values() for c in v[2:]]
    need = max(zb.zsm_prefill_workspace_bytes(c.h, prompt_len, window) for c in caches)
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    for layer in range(n_layers):
        K, V, Qw = wl.prompt(w, layer, dev, u)
        for c in caches:
            c.prefill(layer, K, V, Qw, ws)
    err = {r: [0.0, 0.0] for r in ratios}
    for s in range(steps):
        q, k, v = wl.decode_inputs(w, s, dev, u)
        o_full = ref.step(q, k, v)
        den = o_full.norm(dim=-1).clamp_min(1e-30)
        for r, (_, _, cm, ce) in cands.items():
            err[r][0] += float(((cm.step(q, k, v) - o_full).norm(dim=-1) / den).mean())
            err[r][1] += float(((ce.step(q, k, v) - o_full).norm(dim=-1) / den).mean())
    for c in caches:
        assert zb.zsm_last_device_status(c.h) == 0
        c.close()
    return {r: {"merge": err[r][0] / steps, "evict": err[r][1] / steps,
                "reduction": 1.0 - err[r][0] / err[r][1], "slots": cands[r][0], "B_r": cands[r][1]}
            for r in ratios}


def sweep(ratio=0.1, **kw):
    """The paper's sensitivity axes (App. C.2) through the same kernels, on synthetic data: mean
    relative output error of the merging cache at one cache ratio while one setting varies --
    B_p/B, B_r/(B - B_p), alpha, lambda, and the slot similarity of Eq. (hatr) (raw dot product
    or its cosine form).  Returns {axis: {value: error}}."""
    out = {"tail_ratio": {}, "dense_ratio": {}, "alpha": {}, "lambda": {}, "similarity": {}}
    for name, sim in (("dot", 0), ("cosine", 1)):
        out["similarity"][name] = run(ratios=(ratio,), similarity=sim, **kw)[ratio]["merge"]
    for t in (0.1, 0.3, 0.5, 0.7, 0.9):
        out["tail_ratio"][t] = run(ratios=(ratio,), tail_ratio=t, **kw)[ratio]["merge"]
    for dr in (0.0, 0.01, 0.02, 0.05, 0.1, 0.2):
        r = run(ratios=(ratio,), dense_ratio=dr, **kw)[ratio]
        out["dense_ratio"][dr] = r["merge"] if dr > 0 else r["evict"]
    for al in (0.0, 0.25, 0.5, 0.75, 1.0):
        out["alpha"][al] = run(ratios=(ratio,), alpha=al, **kw)[ratio]["merge"]
    for lm in (0.0, 0.5, 0.9, 0.98, 1.0):
        out["lambda"][lm] = run(ratios=(ratio,), lam=lm, **kw)[ratio]["merge"]
    return out


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--prompt", type=int, default=4096)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--dense-ratio", type=float, default=0.02)
    ap.add_argument("--seed", type=int, default=41)
    ap.add_argument("--sweep", action="store_true", help="vary B_p/B, B_r share, alpha, lambda at 10 %")
    a = ap.parse_args()
    if a.sweep:
        print(json.dumps(sweep(prompt_len=a.prompt, steps=a.steps, seed=a.seed)))
        raise SystemExit(0)
    print(json.dumps(run(prompt_len=a.prompt, steps=a.steps, dense_ratio=a.dense_ratio, seed=a.seed)))
