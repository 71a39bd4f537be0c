"""Host-side checks of the C ABI that need no GPU: the library loads, exports every entry
point the header declares, and its host-only calls behave."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def zb():
    from paper_2503_10714_b200 import build
    build.build()
    from paper_2503_10714_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "zsm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zsm_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(zb):
    names = declared_symbols()
    assert len(names) >= 15
    lib = ctypes.CDLL(zb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/zsm.h but not exported"
    assert sorted(zb.SYMBOLS) == names, "binding and header disagree on the entry points"
    for n in names:
        assert callable(getattr(zb, n)), f"binding lacks {n}"


def test_split_budget_matches_oracle_helper(zb, oracle):
    for B in list(range(1, 300)) + [819, 2700, 5400, 10800, 54000]:
        assert zb.zsm_split_budget(B) == oracle.split_budget(B)
        bp, bc, br = zb.zsm_split_budget(B)
        assert bp + bc + br == B and bp + bc >= 1
    assert zb.zsm_split_budget(100, 0.5, 0.0) == (50, 50, 0)
    assert zb.zsm_split_budget(100, 0.3, 0.05) == oracle.split_budget(100, 0.3, 0.05)
    for bad in [(0, 0.5, 0.02), (10, -0.1, 0.02), (10, 0.5, 1.5)]:
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_split_budget(*bad)
        assert e.value.status == zb.ZSM_ERR_INVALID_ARG


def test_cache_bytes_scales_with_the_budgets(zb):
    def nbytes(B, dtype="f16", L=2, b=3, H=4):
        bp, bc, br = zb.zsm_split_budget(B)
        cfg = zb.make_config(L, b, H, H, 128, dtype, np.full(L * H, bp), np.full(L * H, bc),
                             np.full(L * H, br))
        return zb.zsm_cache_bytes(cfg)
    small, big = nbytes(200), nbytes(2000)
    per_slot = (big - small) / (1800 * 2 * 3 * 4)
    assert 512 <= per_slot <= 560          # 2 x 256-byte rows + score + pos (+ fp32 merged rows)
    assert nbytes(2000, "f32") > 1.9 * big - 2 * small
    # the headline workload: 1024 units x 2700 slots
    bp, bc, br = zb.zsm_split_budget(2700)
    cfg = zb.make_config(32, 1, 32, 32, 128, "f16", np.full(1024, bp), np.full(1024, bc),
                         np.full(1024, br))
    assert 1.40e9 < zb.zsm_cache_bytes(cfg) < 1.50e9


def test_invalid_configs_are_rejected_on_the_host(zb):
    ok = dict(n_layers=1, batch=1, n_q_heads=4, n_kv_heads=2, head_dim=128, dtype="f16",
              budget_p=[4, 4], budget_c=[4, 4], budget_r=[1, 1])
    zb.zsm_cache_bytes(zb.make_config(**ok))
    for patch in [dict(n_layers=0), dict(n_q_heads=3), dict(budget_p=[0, 4], budget_c=[0, 4]),
                  dict(budget_r=[-1, 1]), dict(lam=1.5), dict(alpha=-0.1), dict(head_dim=0)]:
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_cache_bytes(zb.make_config(**{**ok, **patch}))
        assert e.value.status == zb.ZSM_ERR_INVALID_ARG
    assert zb.zsm_status_string(zb.ZSM_ERR_TIMEOUT) == "device-side wait timed out"
    assert zb.zsm_status_string(zb.ZSM_ERR_NO_MEMORY) == "out of host memory"
    assert zb._lib.zsm_selftest_wait_timeout(None, 1000, None) == zb.ZSM_ERR_INVALID_ARG
    # null handles never reach CUDA
    assert zb._lib.zsm_cache_free(None) == zb.ZSM_ERR_INVALID_ARG
    assert zb._lib.zsm_decode_step(None, 0, None, None, None, None, None, None, None) == zb.ZSM_ERR_INVALID_ARG
