"""Pins for the oracle's one-shot prompt compression (score window, selection, merge chain)."""
import numpy as np
import pytest

from naive import causal_attention_matrix, heavy_hitter_stream


def _prompt(rng, T, d, G):
    q, k, v = heavy_hitter_stream(rng, T, d, G, frac=0.04)
    Q = np.ascontiguousarray(q.transpose(1, 0, 2))          # [G][T][d]: query of every position
    return Q, k, v


@pytest.mark.parametrize("G", [1, 2])
@pytest.mark.parametrize("W", [1, 5, 48])
def test_scores_equal_naive_causal_attention(oracle, G, W):
    """Scores of the prompt pass = Eq. (score) unrolled over the last W rows of the naive
    causal attention matrix: s_t = (1/G) sum_g sum_tau lam^(T-1-tau) A_g[tau, t]."""
    rng = np.random.default_rng(4)
    T, d, lam = 48, 8, 0.9
    Q, K, V = _prompt(rng, T, d, G)
    u = oracle.Unit(d, G, 4, 6, 2, lam=lam)
    res = u.prefill_compress(K, V, Qw=Q[:, T - W:, :])
    want = np.zeros(T)
    for g in range(G):
        A = causal_attention_matrix(Q[g], K, 1 / np.sqrt(d))
        for tau in range(T - W, T):
            want += lam ** (T - 1 - tau) * A[tau]
    want /= G
    np.testing.assert_allclose(res.scores, want.astype(np.float32), rtol=2e-7, atol=1e-30)


def test_full_window_matches_decode_recurrence(oracle):
    """With W = T the prompt pass and a token-by-token run through an unbounded cache apply
    the same recurrence; they differ only by the per-step fp32 rounding of the latter."""
    rng = np.random.default_rng(6)
    T, d, G = 64, 8, 2
    Q, K, V = _prompt(rng, T, d, G)
    seq = oracle.Unit(d, G, 8, T, 0)
    for t in range(T):
        seq.decode_step(Q[:, t, :], K[t], V[t])
    pos, sc, _, _ = seq.tokens()
    one = oracle.Unit(d, G, 8, T, 0)
    res = one.prefill_compress(K, V, Qw=Q)
    np.testing.assert_allclose(res.scores[pos], sc, rtol=1e-5)
    assert one.counts() == seq.counts()
    p1, s1, K1, V1 = one.tokens()
    np.testing.assert_array_equal(np.sort(p1), np.sort(pos))
    np.testing.assert_array_equal(K1, K[p1])
    np.testing.assert_array_equal(V1, V[p1])
    assert not res.evicted.any()


def _merge_chain_numpy(K, V, evicted_positions, Br):
    """Eq. (hatr)/(kvr) applied to a stream of tokens, written independently in numpy."""
    Kr, Vr, w, targets = [], [], [], []
    for t in evicted_positions:
        if Br == 0:
            targets.append(-1)
        elif len(Kr) < Br:
            Kr.append(K[t].copy()), Vr.append(V[t].copy()), w.append(1)
            targets.append(-2)
        else:
            dots = np.array([np.float32(kr @ K[t]) for kr in Kr])
            r = int(np.argmax(dots))
            Kr[r] = (w[r] * Kr[r] + K[t]) / (w[r] + 1)
            Vr[r] = (w[r] * Vr[r] + V[t]) / (w[r] + 1)
            w[r] += 1
            targets.append(r)
    return Kr, Vr, w, targets


@pytest.mark.parametrize("budgets", [(8, 10, 3), (0, 12, 2), (10, 0, 4), (6, 9, 0), (5, 7, 1), (40, 100, 5), (3, 4, 60)])
def test_selection_and_merge_chain_brute_force(oracle, budgets):
    """Latest B_p positions kept; of the rest the B_c highest (score, position) kept (sorted
    brute force); the others merged in ascending position by fill-or-merge; conservation."""
    Bp, Bc, Br = budgets
    rng = np.random.default_rng(12)
    T, d, G = 96, 8, 1
    Q, K, V = _prompt(rng, T, d, G)
    u = oracle.Unit(d, G, Bp, Bc, Br)
    res = u.prefill_compress(K, V, Qw=Q[:, T - 16:, :])
    n_prox = min(T, Bp)
    cand = list(range(T - n_prox))
    order = sorted(cand, key=lambda t: (res.scores[t], t))
    n_ev = max(0, len(cand) - Bc)
    ev = sorted(order[:n_ev])
    assert np.flatnonzero(res.evicted).tolist() == ev
    assert res.report.n_evicted == n_ev
    Kr, Vr, w, targets = _merge_chain_numpy(K, V, ev, Br)
    assert res.targets.tolist() == targets
    oKr, oVr, ow = u.residual()
    assert ow.tolist() == w
    if w:
        np.testing.assert_allclose(oKr, np.stack(Kr), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(oVr, np.stack(Vr), rtol=1e-12, atol=1e-14)
    pos, sc, Kt, Vt = u.tokens()
    assert sorted(pos.tolist()) == sorted(set(range(T)) - set(ev))
    np.testing.assert_array_equal(sc, res.scores[pos])
    np.testing.assert_array_equal(Kt, K[pos])
    np.testing.assert_array_equal(Vt, V[pos])
    np_, nc, nr, Tn = u.counts()
    assert np_ == n_prox and nc == len(cand) - n_ev and nr == min(Br, n_ev) and Tn == T
    if Br >= 1:
        assert len(pos) + int(ow.sum()) == T
        members = [[] for _ in w]
        for t, r in zip(ev, targets):
            members[len([x for x in targets[: ev.index(t)] if x == -2]) if r == -2 else r].append(t)
        for r, m in enumerate(members):
            np.testing.assert_allclose(ow[r] * oKr[r], K[m].sum(axis=0), rtol=1e-10, atol=1e-10)
            np.testing.assert_allclose(ow[r] * oVr[r], V[m].sum(axis=0), rtol=1e-10, atol=1e-10)


def test_selection_ties_evict_lower_position_first(oracle):
    """Given scores with exact duplicates, equal scores lose the lower position first."""
    T, d = 12, 4
    rng = np.random.default_rng(0)
    K, V = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    s = np.array([5, 1, 1, 1, 3, 1, 2, 9, 9, 9, 9, 9], dtype=np.float32)
    u = oracle.Unit(d, 1, Bp=2, Bc=5, Br=1)
    res = u.prefill_compress(K, V, scores=s)
    # candidates 0..9, evict 5: the four 1s are {1,2,3,5}; all go, then the 2 at position 6
    assert np.flatnonzero(res.evicted).tolist() == [1, 2, 3, 5, 6]
    u2 = oracle.Unit(d, 1, Bp=2, Bc=7, Br=1)
    res2 = u2.prefill_compress(K, V, scores=s)
    # evict 3 of the four 1s: the three lowest positions
    assert np.flatnonzero(res2.evicted).tolist() == [1, 2, 3]


def test_prompt_shorter_than_budget_is_kept_whole(oracle):
    rng = np.random.default_rng(2)
    T, d = 10, 4
    Q, K, V = _prompt(rng, T, d, 1)
    for Bp, Bc in [(16, 16), (4, 6), (10, 1), (3, 20)]:
        u = oracle.Unit(d, 1, Bp, Bc, 2)
        res = u.prefill_compress(K, V, Qw=Q[:, -4:, :])
        assert not res.evicted.any() and u.counts() == (min(T, Bp), T - min(T, Bp), 0, T)


def test_decode_continues_after_prefill(oracle):
    """After the one-shot compression the unit is an ordinary Algorithm 1 state: the next
    token gets position T, occupancy stays bounded and the laws of the online path hold."""
    rng = np.random.default_rng(13)
    T, d, G = 80, 8, 2
    Q, K, V = _prompt(rng, T + 20, d, G)
    u = oracle.Unit(d, G, 6, 8, 2)
    u.prefill_compress(K[:T], V[:T], Qw=Q[:, T - 8:T, :])
    for t in range(T, T + 20):
        _, rep = u.decode_step(Q[:, t, :], K[t], V[t])
        assert rep.victim_pos >= 0 and rep.merge_slot >= 0
        pos, _, _, _ = u.tokens()
        assert sorted(pos.tolist())[-6:] == list(range(t - 5, t + 1))
        _, _, w = u.residual()
        assert len(pos) + int(w.sum()) == t + 1


def test_prefill_hints(oracle):
    """A hinted eviction set that swaps two near-equal boundary tokens is taken; one that
    swaps distant tokens is refused and counted."""
    T, d = 16, 4
    rng = np.random.default_rng(3)
    K, V = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    s = np.linspace(1.0, 2.0, T).astype(np.float32)
    s[5] = np.float32(1.38)
    s[6] = np.nextafter(np.float32(1.38), np.float32(2))
    u = oracle.Unit(d, 1, Bp=2, Bc=8, Br=1)
    own = u.prefill_compress(K, V, scores=s)
    assert own.evicted[5] and not own.evicted[6]
    swapped = own.evicted.copy()
    swapped[5], swapped[6] = False, True
    r = u.prefill_compress(K, V, scores=s, hint_evicted=swapped, tol=1e-4)
    assert r.report.n_near_tie_sel == 1 and r.report.n_mismatch_sel == 0
    assert r.evicted.tolist() == swapped.tolist()
    far = own.evicted.copy()
    far[0], far[13] = False, True
    r = u.prefill_compress(K, V, scores=s, hint_evicted=far, tol=1e-4)
    assert r.report.n_mismatch_sel == 2 and r.evicted.tolist() == own.evicted.tolist()
    # merge-target hints: own targets are accepted silently, a wrong one is refused
    u3 = oracle.Unit(d, 1, Bp=2, Bc=4, Br=2)
    own3 = u3.prefill_compress(K, V, scores=s)
    r = u3.prefill_compress(K, V, scores=s, hint_targets=own3.targets, tol=1e-6)
    assert r.report.n_near_tie_merge == 0 and r.report.n_mismatch_merge == 0
    bad = own3.targets.copy()
    bad[-1] = 1 - bad[-1]
    r = u3.prefill_compress(K, V, scores=s, hint_targets=bad, tol=1e-9)
    assert r.report.n_mismatch_merge == 1 and r.targets.tolist() == own3.targets.tolist()


@pytest.mark.parametrize("Br", [2, 9, 40])
def test_planted_merge_ties_in_the_prompt_chain(oracle, Br):
    """Exact ties of Eq. (hatr) planted in the prompt's evicted stream (tie_streams): each
    tie token goes to the lower slot of its pair, and the whole chain equals the independent
    numpy chain (np.argmax returns the first maximum)."""
    from tie_streams import planted_prompt
    d, Bp, Bc = 16, 3, 5
    rng = np.random.default_rng(60 + Br)
    K, V, s, n_ev, want = planted_prompt(rng, d, Bp, Bc, Br, n_more=30)
    u = oracle.Unit(d, 1, Bp, Bc, Br)
    res = u.prefill_compress(K, V, scores=s)
    assert np.flatnonzero(res.evicted).tolist() == list(range(n_ev))
    assert res.targets[:Br].tolist() == [-2] * Br
    assert res.targets[Br:Br + len(want)].tolist() == want
    assert res.report.min_merge_gap == 0.0
    _, _, _, targets = _merge_chain_numpy(K, V, list(range(n_ev)), Br)
    assert res.targets.tolist() == targets
