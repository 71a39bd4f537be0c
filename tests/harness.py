"""Shared machinery of the GPU parity tests: drives the C ABI through the binding and
the oracle side by side on the same seeded inputs.

Selection protocol.  The two integer decisions of a step (which token is evicted,
which merged slot absorbs it) are taken in fp32 on both sides, but the fp32 values
come from different summation orders and exponential routines, so a choice between
two candidates closer than the arithmetic can resolve is not unique.  The oracle is
therefore told the GPU's choice as a hint: it takes it only if it is its own choice or
lies within HINT_TOL (relative) of it -- a "near tie", counted and reported --
and otherwise keeps its own and flags a mismatch, which fails the test.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

import workloads as wl

HINT_TOL = 1e-4
OUT_TOL = {"f32": (1e-5, 1e-4), "f16": (2e-3, 1e-2), "bf16": (2e-3, 1e-2)}  # (atol, rtol)
SCORE_RTOL = 1e-4
RESIDUAL_TOL = (1e-4, 1e-4)  # merged rows are fp32 masters on the GPU, fp64 in the oracle


def split_budgets(zb, totals: np.ndarray):
    """Per-head (B_p, B_c, B_r) arrays from total slots with the paper's recommended ratios."""
    bp = np.zeros_like(totals)
    bc = np.zeros_like(totals)
    br = np.zeros_like(totals)
    for idx in np.ndindex(totals.shape):
        bp[idx], bc[idx], br[idx] = zb.zsm_split_budget(int(totals[idx]))
    return bp, bc, br


class GpuCache:
    """One zsm cache with its device buffer; thin convenience over the binding."""

    def __init__(self, zb, w: wl.Workload, bp, bc, br, lam=0.98, alpha=1.0, scale=0.0, **tune):
        self.zb, self.w = zb, w
        self.bp = np.asarray(bp, np.int32).reshape(w.n_layers, w.n_kv_heads)
        self.bc = np.asarray(bc, np.int32).reshape(w.n_layers, w.n_kv_heads)
        self.br = np.asarray(br, np.int32).reshape(w.n_layers, w.n_kv_heads)
        self.lam, self.alpha = lam, alpha
        self.similarity = int(tune.get("similarity", 0))
        self.cfg = zb.make_config(w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim,
                                  w.dtype, self.bp, self.bc, self.br, lam, alpha, scale, **tune)
        nbytes = zb.zsm_cache_bytes(self.cfg)
        self.buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        assert self.buf.data_ptr() % 256 == 0
        self.h = zb.zsm_cache_create(self.cfg, self.buf)
        self.ws = None
        dev = "cuda"
        self.out_all = torch.empty(w.n_layers, w.batch, w.n_q_heads, w.head_dim,
                                   dtype=w.torch_dtype, device=dev)
        self.vic_all = torch.empty(w.n_layers, w.batch, w.n_kv_heads, dtype=torch.int32, device=dev)
        self.slot_all = torch.empty_like(self.vic_all)

    def close(self):
        if self.h is not None:
            self.zb.zsm_cache_free(self.h)
            self.h = None

    def decode(self, q, k, v, layer=-1):
        """q [L,b,Hq,d], k/v [L,b,Hkv,d] device tensors.  layer=-1: one launch for all layers;
        layer='each': one launch per layer.  Returns (out, victim_pos, merge_slot) views."""
        zb = self.zb
        if layer == -1:
            zb.zsm_decode_step(self.h, -1, q, k, v, self.out_all, self.vic_all, self.slot_all)
        else:
            layers = range(self.w.n_layers) if layer == "each" else [layer]
            for l in layers:
                zb.zsm_decode_step(self.h, l, q[l], k[l], v[l], self.out_all[l], self.vic_all[l],
                                   self.slot_all[l])
        return self.out_all, self.vic_all, self.slot_all

    def prefill(self, layer, K, V, Qw=None, scores=None, dbg=True):
        zb, w = self.zb, self.w
        T = K.shape[2]
        W = 0 if Qw is None else Qw.shape[2]
        need = zb.zsm_prefill_workspace_bytes(self.h, T, W)
        if self.ws is None or self.ws.numel() < need:
            self.ws = None
            self.ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        d = {}
        if dbg:
            d["scores"] = torch.empty(w.batch, w.n_kv_heads, T, dtype=torch.float32, device="cuda")
            d["evicted"] = torch.zeros(w.batch, w.n_kv_heads, T, dtype=torch.uint8, device="cuda")
            d["targets"] = torch.full((w.batch, w.n_kv_heads, T), -9, dtype=torch.int32, device="cuda")
        zb.zsm_prefill_compress(self.h, layer, K, V, Qw, scores, T, W, self.ws, d.get("scores"),
                                d.get("evicted"), d.get("targets"))
        return d

    def export(self, layer, b, h):
        return self.zb.zsm_cache_export_unit(self.h, layer, b, h, self.w.head_dim)

    def status(self):
        return self.zb.zsm_last_device_status(self.h)


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


@dataclass
class ParityStats:
    steps: int = 0
    selections: int = 0
    merges: int = 0
    victim_near_ties: int = 0
    merge_near_ties: int = 0
    exact_tie_breaches: int = 0
    max_out_err: float = 0.0
    max_score_rel: float = 0.0
    max_res_err: float = 0.0
    notes: list = field(default_factory=list)


def assert_close(got, want, atol, rtol, what):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    err = np.abs(got - want)
    bad = err > atol + rtol * np.abs(want)
    if bad.any():
        i = np.unravel_index(np.argmax(err - (atol + rtol * np.abs(want))), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside atol={atol} rtol={rtol}; "
                             f"worst at {i}: got {got[i]!r} want {want[i]!r}")
    return float(err.max()) if err.size else 0.0


def oracle_unit_for(oracle, cache: GpuCache, layer, h):
    w = cache.w
    return oracle.Unit(w.head_dim, w.group, int(cache.bp[layer, h]), int(cache.bc[layer, h]),
                       int(cache.br[layer, h]), lam=float(np.float32(cache.lam)),
                       alpha=float(np.float32(cache.alpha)), cosine=bool(cache.similarity))


def oracle_step_check(unit, q, k, v, out_gpu, vic_gpu, slot_gpu, dtype, stats: ParityStats, tag=""):
    """One oracle step hinted with the GPU's choices; asserts selection and output parity."""
    o, rep = unit.decode_step(q, k, v, hint_victim=int(vic_gpu),
                              hint_slot=int(slot_gpu) if slot_gpu >= 0 else -1, tol=HINT_TOL)
    assert not rep.victim_mismatch, (
        f"{tag}: GPU evicted position {vic_gpu}, oracle {rep.victim_own_pos} "
        f"(runner-up {rep.victim_runner_pos}, gap {rep.victim_gap:.3e})")
    assert not rep.merge_mismatch, (
        f"{tag}: GPU merged into slot {slot_gpu}, oracle {rep.merge_own_slot} "
        f"(runner-up {rep.merge_runner_slot}, gap {rep.merge_gap:.3e})")
    assert rep.victim_pos == vic_gpu, f"{tag}: victim {vic_gpu} vs oracle {rep.victim_pos}"
    assert rep.merge_slot == slot_gpu, f"{tag}: merge slot {slot_gpu} vs oracle {rep.merge_slot}"
    stats.steps += 1
    stats.selections += rep.victim_pos >= 0
    stats.merges += rep.merge_slot >= 0
    stats.victim_near_ties += rep.victim_near_tie
    stats.merge_near_ties += rep.merge_near_tie
    stats.exact_tie_breaches += rep.victim_exact_tie + rep.merge_exact_tie
    atol, rtol = OUT_TOL[dtype]
    stats.max_out_err = max(stats.max_out_err, assert_close(out_gpu, o, atol, rtol, f"{tag}: output"))
    return rep


def state_check(unit, st: dict, stats: ParityStats, tag=""):
    """Exported GPU unit state against the oracle's lists, matched by position."""
    np_, nc, nr, T = unit.counts()
    assert (st["n_live"], st["n_res"], st["T"]) == (np_ + nc, nr, T), \
        f"{tag}: counters {(st['n_live'], st['n_res'], st['T'])} vs oracle {(np_ + nc, nr, T)}"
    pos, sc, K, V = unit.tokens()
    go, oo = np.argsort(st["pos"]), np.argsort(pos)
    np.testing.assert_array_equal(st["pos"][go], pos[oo], err_msg=f"{tag}: retained positions")
    np.testing.assert_array_equal(st["K"][go].astype(np.float64), K[oo], err_msg=f"{tag}: K rows")
    np.testing.assert_array_equal(st["V"][go].astype(np.float64), V[oo], err_msg=f"{tag}: V rows")
    rel = np.abs(st["score"][go].astype(np.float64) - sc[oo]) / np.maximum(np.abs(sc[oo]), 1e-30)
    if rel.size:
        stats.max_score_rel = max(stats.max_score_rel, float(rel.max()))
        assert rel.max() <= SCORE_RTOL, f"{tag}: score relative error {rel.max():.3e}"
    Kr, Vr, w = unit.residual()
    np.testing.assert_array_equal(st["w"], w, err_msg=f"{tag}: fusion counts")
    if nr:
        a, r = RESIDUAL_TOL
        e1 = assert_close(st["Kr"], Kr, a, r, f"{tag}: merged keys")
        e2 = assert_close(st["Vr"], Vr, a, r, f"{tag}: merged values")
        stats.max_res_err = max(stats.max_res_err, e1, e2)


def prefill_check(oracle, cache: GpuCache, layer, b, h, K, V, Qw, dbg, stats: ParityStats,
                  scores_given=None, tag=""):
    """Oracle prompt compression of unit (layer, b, h), hinted with the GPU's eviction set
    and merge targets; asserts scores, selection, targets and the resulting state."""
    w = cache.w
    G = w.group
    unit = oracle_unit_for(oracle, cache, layer, h)
    ev_gpu = dbg["evicted"][b, h].cpu().numpy().astype(bool)
    n_ev = int(ev_gpu.sum())
    tg_gpu = dbg["targets"][b, h, :n_ev].cpu().numpy()
    hint_t = np.where(tg_gpu >= 0, tg_gpu, -1).astype(np.int32)
    kw = dict(hint_evicted=ev_gpu, hint_targets=hint_t, tol=HINT_TOL)
    if scores_given is None:
        res = unit.prefill_compress(f64(K[b, h]), f64(V[b, h]), Qw=f64(Qw[b, h * G:(h + 1) * G]), **kw)
        s_gpu = dbg["scores"][b, h].cpu().numpy().astype(np.float64)
        rel = np.abs(s_gpu - res.scores) / np.maximum(np.abs(res.scores.astype(np.float64)), 1e-30)
        stats.max_score_rel = max(stats.max_score_rel, float(rel.max()))
        bad = np.flatnonzero(rel > SCORE_RTOL)
        assert bad.size == 0, (f"{tag}: prompt score relative error {rel.max():.3e} at {bad.size} positions, "
                               f"first {bad[:6].tolist()}, last {bad[-3:].tolist()}, 128-position chunks "
                               f"{sorted(set((bad // 128).tolist()))[:24]}")
    else:
        res = unit.prefill_compress(f64(K[b, h]), f64(V[b, h]), scores=scores_given, **kw)
    r = res.report
    assert r.n_mismatch_sel == 0, f"{tag}: eviction sets differ beyond near ties (gap {r.sel_gap:.3e})"
    assert r.n_mismatch_merge == 0, f"{tag}: merge targets differ beyond near ties (min gap {r.min_merge_gap:.3e})"
    assert r.n_evicted == n_ev, f"{tag}: evicted {n_ev} vs oracle {r.n_evicted}"
    assert r.n_exact_tie_merge == 0, (f"{tag}: {r.n_exact_tie_merge} merge targets were not the lowest "
                                      "slot among exactly equal dot products")
    np.testing.assert_array_equal(res.evicted, ev_gpu, err_msg=f"{tag}: eviction flags")
    np.testing.assert_array_equal(res.targets, tg_gpu, err_msg=f"{tag}: merge targets")
    stats.selections += n_ev
    stats.merges += int((tg_gpu >= 0).sum())
    stats.victim_near_ties += r.n_near_tie_sel
    stats.merge_near_ties += r.n_near_tie_merge
    stats.exact_tie_breaches += r.n_exact_tie_merge
    state_check(unit, cache.export(layer, b, h), stats, tag=tag + " state after prompt pass")
    return unit
