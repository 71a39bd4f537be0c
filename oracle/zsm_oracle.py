"""ctypes front end of the ZSMerge CPU oracle -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
module.  It never touches the CUDA library and is never a fallback for it.

`build()` compiles zsm_oracle.c with gcc (-O2 -fopenmp) into
libzsm_oracle.so beside the source; `Unit` wraps one (layer, sequence,
kv-head) cache of Algorithm 1.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zsm_oracle.c")
_HDR = os.path.join(_HERE, "zsm_oracle.h")
_LIB = os.path.join(_HERE, "libzsm_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its sources."""
    stale = force or not os.path.exists(_LIB)
    if not stale:
        t = os.path.getmtime(_LIB)
        stale = t < os.path.getmtime(_SRC) or t < os.path.getmtime(_HDR)
    if stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Params(C.Structure):
    _fields_ = [("d", C.c_int32), ("G", C.c_int32), ("Bp", C.c_int32), ("Bc", C.c_int32),
                ("Br", C.c_int32), ("lam", C.c_double), ("alpha", C.c_double),
                ("scale", C.c_double), ("cosine", C.c_int32)]


class _Hint(C.Structure):
    _fields_ = [("victim_pos", C.c_int32), ("merge_slot", C.c_int32), ("tol", C.c_double)]


class StepReport(C.Structure):
    _fields_ = [("victim_pos", C.c_int32), ("victim_own_pos", C.c_int32),
                ("victim_runner_pos", C.c_int32), ("victim_gap", C.c_double),
                ("merge_slot", C.c_int32), ("merge_own_slot", C.c_int32),
                ("merge_runner_slot", C.c_int32), ("merge_gap", C.c_double),
                ("victim_near_tie", C.c_int32), ("merge_near_tie", C.c_int32),
                ("victim_mismatch", C.c_int32), ("merge_mismatch", C.c_int32),
                ("victim_exact_tie", C.c_int32), ("merge_exact_tie", C.c_int32)]


class PrefillReport(C.Structure):
    _fields_ = [("n_evicted", C.c_int32), ("n_near_tie_sel", C.c_int32),
                ("n_mismatch_sel", C.c_int32), ("n_near_tie_merge", C.c_int32),
                ("n_mismatch_merge", C.c_int32), ("min_merge_gap", C.c_double),
                ("sel_gap", C.c_double), ("n_exact_tie_merge", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, dp = C.c_void_p, C.POINTER(C.c_double)
        L.zso_unit_new.restype = vp
        L.zso_unit_new.argtypes = [C.POINTER(_Params)]
        L.zso_unit_free.argtypes = [vp]
        L.zso_decode_step.restype = C.c_int
        L.zso_decode_step.argtypes = [vp, dp, dp, dp, dp, C.POINTER(_Hint),
                                      C.POINTER(StepReport)]
        L.zso_prefill_compress.restype = C.c_int
        L.zso_prefill_compress.argtypes = [vp, dp, dp, dp, C.POINTER(C.c_float), C.c_int32,
                                           C.c_int32, C.POINTER(C.c_uint8),
                                           C.POINTER(C.c_int32), C.c_double,
                                           C.POINTER(C.c_float), C.POINTER(C.c_uint8),
                                           C.POINTER(C.c_int32), C.POINTER(PrefillReport)]
        L.zso_counts.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                 C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
        L.zso_export_tokens.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_float), dp, dp]
        L.zso_export_residual.argtypes = [vp, dp, dp, C.POINTER(C.c_uint32)]
        L.zso_last_attention.restype = C.c_int32
        L.zso_last_attention.argtypes = [vp, dp, C.POINTER(C.c_int64)]
        L.zso_decode_step_batch.restype = C.c_int
        L.zso_decode_step_batch.argtypes = [C.POINTER(vp), C.c_int32, dp, dp, dp, dp]
        L.zso_split_budget.restype = C.c_int
        L.zso_split_budget.argtypes = [C.c_int32, C.c_double, C.c_double,
                                       C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                       C.POINTER(C.c_int32)]
        _lib = L
    return _lib


def _dp(a):
    return None if a is None else a.ctypes.data_as(C.POINTER(C.c_double))


def _f64(a, shape=None):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def split_budget(B: int, tail_ratio: float = 0.5, dense_ratio: float = 0.02):
    """(B_p, B_c, B_r) from the two ratios of App. C.2."""
    bp, bc, br = C.c_int32(), C.c_int32(), C.c_int32()
    rc = lib().zso_split_budget(int(B), float(tail_ratio), float(dense_ratio), C.byref(bp),
                                C.byref(bc), C.byref(br))
    if rc != 0:
        raise ValueError("bad budget arguments")
    return bp.value, bc.value, br.value


@dataclass
class PrefillResult:
    scores: np.ndarray    # [T] fp32
    evicted: np.ndarray   # [T] bool
    targets: np.ndarray   # [n_evicted] int32: slot per evicted token (-2 fill, -1 dropped)
    report: PrefillReport


class Unit:
    """One (layer, sequence, kv-head) compressed cache, Algorithm 1 in fp64."""

    def __init__(self, d, G, Bp, Bc, Br, lam=0.98, alpha=1.0, scale=None, cosine=False):
        self.d, self.G, self.Bp, self.Bc, self.Br = int(d), int(G), int(Bp), int(Bc), int(Br)
        p = _Params(self.d, self.G, self.Bp, self.Bc, self.Br, float(lam), float(alpha),
                    float(scale) if scale else 1.0 / np.sqrt(float(d)), 1 if cosine else 0)
        self._h = lib().zso_unit_new(C.byref(p))
        if not self._h:
            raise ValueError("invalid oracle unit parameters")

    def close(self):
        if getattr(self, "_h", None):
            lib().zso_unit_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- Algorithm 1 -------------------------------------------------------
    def decode_step(self, q, k_new, v_new, hint_victim=-1, hint_slot=-1, tol=0.0):
        """Returns (out [G][d] fp64, StepReport)."""
        q = _f64(q, (self.G, self.d))
        k = _f64(k_new, (self.d,))
        v = _f64(v_new, (self.d,))
        out = np.empty((self.G, self.d), dtype=np.float64)
        rep = StepReport()
        hint = None
        if hint_victim >= 0 or hint_slot >= 0:
            hint = C.byref(_Hint(int(hint_victim), int(hint_slot), float(tol)))
        rc = lib().zso_decode_step(self._h, _dp(q), _dp(k), _dp(v), _dp(out), hint,
                                   C.byref(rep))
        if rc != 0:
            raise RuntimeError("zso_decode_step failed")
        return out, rep

    def prefill_compress(self, K, V, Qw=None, scores=None, hint_evicted=None,
                         hint_targets=None, tol=0.0) -> PrefillResult:
        K = _f64(K)
        V = _f64(V)
        T = K.shape[0]
        assert K.shape == (T, self.d) and V.shape == (T, self.d)
        W = 0
        qp = None
        sp = None
        if Qw is not None:
            Qw = _f64(Qw)
            assert Qw.ndim == 3 and Qw.shape[0] == self.G and Qw.shape[2] == self.d
            W = Qw.shape[1]
            qp = _dp(Qw)
        else:
            scores = np.ascontiguousarray(np.asarray(scores, dtype=np.float32))
            assert scores.shape == (T,)
            sp = scores.ctypes.data_as(C.POINTER(C.c_float))
        he = None
        if hint_evicted is not None:
            hint_evicted = np.ascontiguousarray(np.asarray(hint_evicted, dtype=np.uint8))
            assert hint_evicted.shape == (T,)
            he = hint_evicted.ctypes.data_as(C.POINTER(C.c_uint8))
        ht = None
        if hint_targets is not None:
            hint_targets = np.ascontiguousarray(np.asarray(hint_targets, dtype=np.int32))
            ht = hint_targets.ctypes.data_as(C.POINTER(C.c_int32))
        s_out = np.empty(T, dtype=np.float32)
        e_out = np.empty(T, dtype=np.uint8)
        t_out = np.full(T, -1, dtype=np.int32)
        rep = PrefillReport()
        rc = lib().zso_prefill_compress(
            self._h, _dp(K), _dp(V), qp, sp, T, W, he, ht, float(tol),
            s_out.ctypes.data_as(C.POINTER(C.c_float)),
            e_out.ctypes.data_as(C.POINTER(C.c_uint8)),
            t_out.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(rep))
        if rc != 0:
            raise RuntimeError("zso_prefill_compress failed")
        return PrefillResult(s_out, e_out.astype(bool), t_out[:rep.n_evicted].copy(), rep)

    # -- inspection --------------------------------------------------------
    def counts(self):
        np_, nc, nr, T = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int64()
        lib().zso_counts(self._h, C.byref(np_), C.byref(nc), C.byref(nr), C.byref(T))
        return np_.value, nc.value, nr.value, T.value

    def tokens(self):
        """(pos [n], score [n] fp32, K [n][d], V [n][d]); K_p (oldest first) then K_c."""
        np_, nc, _, _ = self.counts()
        n = np_ + nc
        pos = np.empty(n, dtype=np.int32)
        sc = np.empty(n, dtype=np.float32)
        K = np.empty((n, self.d), dtype=np.float64)
        V = np.empty((n, self.d), dtype=np.float64)
        lib().zso_export_tokens(self._h, pos.ctypes.data_as(C.POINTER(C.c_int32)),
                                sc.ctypes.data_as(C.POINTER(C.c_float)), _dp(K), _dp(V))
        return pos, sc, K, V

    def residual(self):
        """(Kr [nr][d], Vr [nr][d], w [nr])."""
        _, _, nr, _ = self.counts()
        Kr = np.empty((nr, self.d), dtype=np.float64)
        Vr = np.empty((nr, self.d), dtype=np.float64)
        w = np.empty(nr, dtype=np.uint32)
        lib().zso_export_residual(self._h, _dp(Kr), _dp(Vr),
                                  w.ctypes.data_as(C.POINTER(C.c_uint32)))
        return Kr, Vr, w

    def last_attention(self):
        """(a [G][n], id [n]): id >= 0 is a token position, -(r+1) residual slot r."""
        n = lib().zso_last_attention(self._h, None, None)
        a = np.empty((self.G, n), dtype=np.float64)
        ids = np.empty(n, dtype=np.int64)
        lib().zso_last_attention(self._h, _dp(a), ids.ctypes.data_as(C.POINTER(C.c_int64)))
        return a, ids


def decode_step_batch(units, q, k_new, v_new):
    """Algorithm 1 over independent units with OpenMP; returns (out, threads used)."""
    n = len(units)
    G, d = units[0].G, units[0].d
    q = _f64(q, (n, G, d))
    k = _f64(k_new, (n, d))
    v = _f64(v_new, (n, d))
    out = np.empty((n, G, d), dtype=np.float64)
    arr = (C.c_void_p * n)(*[u._h for u in units])
    threads = lib().zso_decode_step_batch(arr, n, _dp(q), _dp(k), _dp(v), _dp(out))
    return out, threads
