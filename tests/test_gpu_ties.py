"""Exact ties on the GPU.  The two integer decisions of a step have tie rules -- the evicted
token is the lowest position among equal scores (Alg. 1), the merged slot the lowest slot
among equal dot products (Eq. (hatr)) -- that random data never exercises.  These tests feed
constructed ties (tie_streams: small integers, exact in every dtype and summation order)
through the C ABI to every kernel that takes such a decision: the fused decode kernel in its
paired and wide launch forms, the split form, and each form of the prompt's merge chain."""
import numpy as np
import pytest
import torch

import workloads as wl
from harness import (GpuCache, ParityStats, f64, oracle_step_check, oracle_unit_for, prefill_check,
                     state_check)
from tie_streams import planted_prompt, tie_tokens

pytestmark = pytest.mark.gpu

# how the decode step is launched: the library's own choice for one unit is the split form (a
# cluster of CTAs); tune_split = 1 gives the fused kernel, one CTA per SM ("wide"); asking for
# two CTAs per SM gives the paired form the all-layer launch of a large model uses
FORMS = {"split": dict(), "wide": dict(tune_split=1), "paired": dict(tune_ctas_per_sm=2)}
TORCH = {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}


@pytest.fixture(scope="module")
def zb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import binding
    return binding


@pytest.mark.parametrize("form", list(FORMS))
def test_exact_score_ties_resolve_by_position(zb, form):
    """Bit-identical tokens give bit-identical scores on the GPU too: the evicted one must be
    the lowest position among the minima (lam = 0: the score is the last attention weight)."""
    w = wl.Workload("ties", 1, 1, 1, 1, 64, "f32", 0, 0, 0, None, 14)
    cache = GpuCache(zb, w, [[1]], [[2]], [[0]], lam=0.0, **FORMS[form])
    try:
        def tok(x):
            t = torch.zeros(1, 1, 1, 64)
            t[..., 0] = x
            return t.cuda()
        q, ones = tok(1.0), torch.ones(1, 1, 1, 64).cuda()
        victims = []
        for x in [1.0, 1.0, 5.0, 5.0, 5.0]:
            _, vic, _ = cache.decode(q, tok(x), ones)
            victims.append(int(vic.cpu()[0, 0, 0]))
        assert victims == [-1, -1, -1, 0, 1]
    finally:
        cache.close()


@pytest.mark.parametrize("form", ["wide", "paired"])
@pytest.mark.parametrize("dtype,d,G", [("f16", 128, 1), ("bf16", 128, 4), ("f32", 64, 2)])
def test_many_equal_scores_across_tiles_and_warps(zb, form, dtype, d, G):
    """600 bit-identical tokens fill a pool that spans several tiles and every consumer warp;
    hotter tokens follow.  Each step must evict the lowest remaining position of the 600: the
    minimum over (score, position) has to come out right across lanes, warps and tiles."""
    n_same, n_hot = 600, 40
    w = wl.Workload("ties_many", 1, 1, G, 1, d, dtype, 0, 0, 0, None, 35)
    cache = GpuCache(zb, w, [[1]], [[n_same - 1]], [[0]], lam=0.0, **FORMS[form])
    try:
        def tok(x):
            t = torch.zeros(1, 1, 1, d)
            t[..., 0] = x
            return t.to(TORCH[dtype]).cuda()
        q = torch.zeros(1, 1, G, d)
        q[..., 0] = 1.0
        q = q.to(TORCH[dtype]).cuda()
        vv = torch.ones(1, 1, 1, d).to(TORCH[dtype]).cuda()
        victims = []
        for i in range(n_same + n_hot):
            _, vic, _ = cache.decode(q, tok(1.0 if i < n_same else 6.0), vv)
            victims.append(vic.clone())
        victims = torch.stack(victims).flatten().cpu().tolist()
        assert victims == [-1] * n_same + list(range(n_hot))
        assert cache.status() == 0
    finally:
        cache.close()


@pytest.mark.parametrize("form", list(FORMS))
@pytest.mark.parametrize("Br", [8, 40, 100])
@pytest.mark.parametrize("dtype,d,G", [("f16", 128, 1), ("bf16", 128, 4), ("f32", 64, 1)])
def test_merge_ties_in_the_decode_step(zb, oracle, form, Br, dtype, d, G):
    """Pairs of merged slots with identical keys, or different keys and the same product, one
    at the front and one at the back of the residual pool; the evicted tokens tie exactly
    between the two.  The state comes from the oracle's prompt pass and is imported; with
    lam = 1 and scores spaced far apart the victims are the tie tokens, in order."""
    rng = np.random.default_rng(500 + Br)
    _, want = tie_tokens(Br, d)
    n_tie = len(want)
    Bp, Bc = n_tie + 2, 40
    K, V, s, _, _ = planted_prompt(rng, d, Bp, Bc, Br, n_more=0)
    s[:Br] = 0.25
    s[Br:Br + n_tie] = 10.0 * (1 + np.arange(n_tie))
    s[Br + n_tie:] = 1000.0 + 10.0 * np.arange(len(s) - Br - n_tie)
    w = wl.Workload("merge_ties", 1, 1, G, 1, d, dtype, 0, 0, 0, None, 36)
    cache = GpuCache(zb, w, [[Bp]], [[Bc + n_tie]], [[Br]], lam=1.0, **FORMS[form])
    stats = ParityStats()
    try:
        unit = oracle_unit_for(oracle, cache, 0, 0)
        res = unit.prefill_compress(K, V, scores=s)
        assert res.report.n_evicted == Br
        pos, sc, Kt, Vt = unit.tokens()
        Kr, Vr, wr = unit.residual()
        zb.zsm_cache_import_unit(cache.h, 0, 0, 0, d, dict(K=Kt, V=Vt, score=sc, pos=pos, Kr=Kr, Vr=Vr,
                                                           w=wr, n_live=len(pos), n_res=len(wr),
                                                           T=len(s)))
        g = torch.Generator().manual_seed(9)
        got = []
        for t in range(n_tie):
            q = torch.randn(1, 1, G, d, generator=g).to(TORCH[dtype])
            k = torch.randn(1, 1, 1, d, generator=g).to(TORCH[dtype])
            v = torch.randn(1, 1, 1, d, generator=g).to(TORCH[dtype])
            out, vic, slot = cache.decode(q.cuda(), k.cuda(), v.cuda())
            rep = oracle_step_check(unit, f64(q)[0, 0], f64(k)[0, 0, 0], f64(v)[0, 0, 0], f64(out)[0, 0],
                                    int(vic.cpu()[0, 0, 0]), int(slot.cpu()[0, 0, 0]), dtype, stats,
                                    tag=f"tie step {t}")
            assert rep.victim_pos == Br + t and rep.merge_gap == 0.0
            got.append(int(slot.cpu()[0, 0, 0]))
        assert got == want
        assert stats.exact_tie_breaches == 0 and stats.merge_near_ties == 0
        state_check(unit, cache.export(0, 0, 0), stats, tag="after the tie steps")
        assert cache.status() == 0
    finally:
        cache.close()


# (dtype, head_dim, B_r, sequences x kv heads) -> the form of the merge chain it selects
CHAIN_FORMS = {
    "blocked, one slot per lane": ("f16", 128, 8, (1, 2)),
    "blocked, two slots per lane": ("bf16", 128, 48, (1, 2)),
    "rows in registers, four per thread": ("f16", 128, 100, (1, 2)),
    "shared-memory form": ("f16", 64, 150, (1, 2)),
    "rows in registers, one per thread (fp32)": ("f32", 64, 8, (1, 2)),
    "rows in registers, two per thread (fp32)": ("f32", 64, 48, (1, 2)),
    "one warp per unit": ("bf16", 64, 8, (40, 8)),
}


@pytest.mark.parametrize("form", list(CHAIN_FORMS))
def test_merge_ties_in_the_prompt_chain(zb, oracle, form):
    """The same planted ties inside the prompt's evicted stream, for every form of the merge
    chain: the tie tokens go to the lower slot of their pair, the rest of the chain (200 more
    tokens) and the resulting state match the oracle."""
    dtype, d, Br, (batch, heads) = CHAIN_FORMS[form]
    Bp, Bc = 12, 20
    w = wl.Workload("chain_ties", 1, batch, heads, heads, d, dtype, 0, 0, 0, None, 37)
    Ks, Vs, Ss, wants = [], [], [], []
    for u in range(batch * heads):
        K, V, s, n_ev, want = planted_prompt(np.random.default_rng(700 + u), d, Bp, Bc, Br, n_more=200)
        Ks.append(K), Vs.append(V), Ss.append(s), wants.append(want)
    T = Ks[0].shape[0]
    shape = (batch, heads, T)
    K = torch.from_numpy(np.stack(Ks)).reshape(*shape, d).to(TORCH[dtype])
    V = torch.from_numpy(np.stack(Vs)).reshape(*shape, d).to(TORCH[dtype])
    S = torch.from_numpy(np.stack(Ss)).reshape(*shape)
    cache = GpuCache(zb, w, np.full((1, heads), Bp), np.full((1, heads), Bc), np.full((1, heads), Br))
    stats = ParityStats()
    try:
        dbg = cache.prefill(0, K.cuda(), V.cuda(), None, S.cuda())
        tg = dbg["targets"].cpu().numpy()
        for b in range(batch):
            for h in range(heads):
                want = wants[b * heads + h]
                assert tg[b, h, :Br].tolist() == [-2] * Br
                assert tg[b, h, Br:Br + len(want)].tolist() == want, f"unit {(b, h)}"
                prefill_check(oracle, cache, 0, b, h, K, V, None, dbg, stats,
                              scores_given=S[b, h].numpy(), tag=f"{form} unit {(b, h)}")
        assert cache.status() == 0 and stats.exact_tie_breaches == 0
    finally:
        cache.close()
