"""The seeded input recipe: shapes, dtypes, determinism, heavy-hitter structure."""
import numpy as np
import torch

import workloads as wl


def test_named_workloads_have_the_stated_shapes():
    assert wl.C1.group == 1 and wl.C5.group == 4
    assert wl.C4_5.budget == round(0.05 * wl.C4_5.prompt_len)
    assert wl.C3.budget == round(0.05 * wl.C3.prompt_len)
    b = wl.head_budgets(wl.C5)
    assert b.shape == (32, 8) and b.min() >= 64 and b.max() <= 2048
    assert abs(b.mean() - 0.05 * wl.C5.prompt_len) < 80
    assert (wl.head_budgets(wl.C2) == 205).all()


def test_streams_are_seeded_and_rounded_to_storage_dtype():
    w = wl.C2.replace(prompt_len=64, n_q_heads=4, n_kv_heads=2, window=8)
    K1, V1, Q1 = wl.prompt(w, 0)
    K2, V2, Q2 = wl.prompt(w, 0)
    assert torch.equal(K1, K2) and torch.equal(V1, V2) and torch.equal(Q1, Q2)
    assert K1.dtype == torch.float16 and K1.shape == (1, 2, 64, 128) and Q1.shape == (1, 4, 8, 128)
    q, k, v = wl.decode_inputs(w, 3)
    q2, _, _ = wl.decode_inputs(w, 4)
    assert q.shape == (1, 1, 4, 128) and k.shape == (1, 1, 2, 128) and not torch.equal(q, q2)
    assert not torch.equal(wl.prompt(w.replace(seed=9), 0)[0], K1)


def test_heavy_hitters_sit_along_the_query_direction():
    w = wl.C1.replace(prompt_len=4000)
    u = wl.directions(w)[0]                                   # [H, d]
    K, _, Qw = wl.prompt(w, 0)
    proj = (K[0].double() * u[:, None, :].double()).sum(-1)   # [H, T]
    c = np.sqrt(4 * np.sqrt(w.head_dim))
    heavy = proj > c / 2
    assert heavy[:, 0].all()
    frac = heavy[:, 1:].double().mean().item()
    assert 0.012 < frac < 0.03
    qproj = (Qw[0].double() * u[:, None, :].double()).sum(-1)
    assert abs(qproj.mean().item() - c) < 0.3
