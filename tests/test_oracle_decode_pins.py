"""Pins for the oracle's decode step (Algorithm 1 + Eq. (att_score2)).

Each test holds the oracle to something other than itself: a textbook routine,
a closed form, a theorem of the paper, a conservation law, or an independently
written second formulation.
"""
import os

import numpy as np
import pytest

from naive import heavy_hitter_stream, sdpa_torch, softmax_attention
from pool_form import PoolCache

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def run_stream(unit, q, k, v):
    outs, reps = [], []
    for t in range(k.shape[0]):
        o, r = unit.decode_step(q[t], k[t], v[t])
        outs.append(o)
        reps.append(r)
    return outs, reps


@pytest.mark.parametrize("G", [1, 4])
def test_no_eviction_equals_full_attention(oracle, G):
    """Budget >= context: every step's output is plain softmax attention (Eq. (att_score)),
    checked against a naive numpy routine and against torch's SDPA in fp64.  alpha must
    not matter while every fusion count is 1 (Sec. 3.5: w = 1 for uncompressed tokens)."""
    rng = np.random.default_rng(10 + G)
    n, d = 40, 16
    q, k, v = heavy_hitter_stream(rng, n, d, G)
    for alpha in (1.0, 0.3):
        u = oracle.Unit(d, G, Bp=7, Bc=n, Br=3, alpha=alpha)
        for t in range(n):
            o, rep = u.decode_step(q[t], k[t], v[t])
            ref, _ = softmax_attention(q[t], k[: t + 1], v[: t + 1], 1 / np.sqrt(d))
            np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(o, sdpa_torch(q[t], k[: t + 1], v[: t + 1], 1 / np.sqrt(d)),
                                       rtol=1e-10, atol=1e-12)
            assert rep.victim_pos == -1 and rep.merge_slot == -1
        assert u.counts() == (7, n - 7, 0, n)


def test_custom_scale_is_used(oracle):
    rng = np.random.default_rng(3)
    n, d = 12, 8
    q, k, v = heavy_hitter_stream(rng, n, d, 1)
    u = oracle.Unit(d, 1, 4, n, 0, scale=0.37)
    for t in range(n):
        o, _ = u.decode_step(q[t], k[t], v[t])
        ref, _ = softmax_attention(q[t], k[: t + 1], v[: t + 1], 0.37)
        np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)


def _duplicate_key_stream(rng, n, d, n_keep):
    """n_keep strongly attended tokens first, then fillers that all share one key."""
    e1 = np.zeros(d)
    e1[0] = 1.0
    q = rng.normal(size=(n, 1, d)) * 0.1 + 6.0 * e1
    k = np.empty((n, d))
    k[:n_keep] = rng.normal(size=(n_keep, d)) * 0.1 + 3.0 * e1
    kstar = rng.normal(size=d) * 0.3 - 2.0 * e1
    k[n_keep:] = kstar
    v = rng.normal(size=(n, d))
    return q, k, v


def test_duplicate_key_closed_form(oracle):
    """If every token merged into a slot has the same key, then with alpha = 1 the slot
    contributes w * exp(l) * mean(v) = sum_m exp(l) v_m: the compressed output equals full
    attention exactly.  Pins Eq. (kvr) (count-weighted mean, count increment) together
    with Eq. (att_score2) (the + log w term)."""
    rng = np.random.default_rng(5)
    n, d = 60, 8
    q, k, v = _duplicate_key_stream(rng, n, d, n_keep=3)
    u = oracle.Unit(d, 1, Bp=2, Bc=3, Br=1, alpha=1.0)
    n_merged = 0
    for t in range(n):
        o, rep = u.decode_step(q[t], k[t], v[t])
        ref, _ = softmax_attention(q[t], k[: t + 1], v[: t + 1], 1 / np.sqrt(d))
        np.testing.assert_allclose(o, ref, rtol=1e-11, atol=1e-13)
        if rep.victim_pos >= 0:
            assert rep.victim_pos >= 3, "a keeper was evicted: the construction is broken"
            n_merged += 1
    assert n_merged == n - 5
    _, _, w = u.residual()
    assert w.tolist() == [n - 5]


def test_duplicate_key_needs_alpha_one(oracle):
    """The closed form above must break for alpha != 1 -- the pin is sensitive to the term."""
    rng = np.random.default_rng(5)
    n, d = 30, 8
    q, k, v = _duplicate_key_stream(rng, n, d, n_keep=3)
    u = oracle.Unit(d, 1, Bp=2, Bc=3, Br=1, alpha=0.5)
    worst = 0.0
    for t in range(n):
        o, _ = u.decode_step(q[t], k[t], v[t])
        ref, _ = softmax_attention(q[t], k[: t + 1], v[: t + 1], 1 / np.sqrt(d))
        worst = max(worst, np.abs(o - ref).max())
    assert worst > 1e-4


@pytest.mark.parametrize("alpha", [0.0, 0.5, 1.0])
@pytest.mark.parametrize("G", [1, 2])
def test_theorem_1(oracle, alpha, G):
    """Theorem 1: for every uncompressed token the compensated weight is at least the weight
    full attention over the whole history would give it (alpha in [0, 1])."""
    rng = np.random.default_rng(100 + G)
    n, d = 120, 16
    q, k, v = heavy_hitter_stream(rng, n, d, G)
    u = oracle.Unit(d, G, Bp=6, Bc=8, Br=2, alpha=alpha)
    checked = 0
    for t in range(n):
        u.decode_step(q[t], k[t], v[t])
        a_hat, ids = u.last_attention()
        _, a_full = softmax_attention(q[t], k[: t + 1], v[: t + 1], 1 / np.sqrt(d))
        for j, pid in enumerate(ids):
            if pid >= 0:
                assert np.all(a_hat[:, j] >= a_full[:, pid] - 1e-15)
                checked += 1
        np.testing.assert_allclose(a_hat.sum(axis=1), 1.0, rtol=1e-12)
    assert checked > n


@pytest.mark.parametrize("budgets", [(6, 8, 2), (3, 4, 2), (1, 1, 1), (0, 5, 3), (5, 0, 2), (4, 6, 0)])
def test_conservation_and_occupancy(oracle, budgets):
    """Eq. (kvr) implies w_r k_r = sum of the keys folded into slot r (same for values);
    with B_r >= 1, #uncompressed + sum_r w_r = T; the lists never exceed their budgets and
    the latest B_p positions are always present (Sec. 3.2)."""
    Bp, Bc, Br = budgets
    rng = np.random.default_rng(7)
    n, d, G = 90, 12, 2
    q, k, v = heavy_hitter_stream(rng, n, d, G)
    u = oracle.Unit(d, G, Bp, Bc, Br)
    members = []
    for t in range(n):
        _, rep = u.decode_step(q[t], k[t], v[t])
        if rep.merge_slot == -2:
            members.append([rep.victim_pos])
        elif rep.merge_slot >= 0:
            members[rep.merge_slot].append(rep.victim_pos)
        np_, nc, nr, T = u.counts()
        assert np_ <= Bp and nc <= Bc and nr <= Br and T == t + 1
        pos, _, K, V = u.tokens()
        assert len(set(pos.tolist())) == len(pos)
        for p in range(max(0, t + 1 - Bp), t + 1):
            assert p in pos
        np.testing.assert_array_equal(K, k[pos])
        np.testing.assert_array_equal(V, v[pos])
        Kr, Vr, w = u.residual()
        assert [len(m) for m in members] == w.tolist()
        for r, m in enumerate(members):
            np.testing.assert_allclose(w[r] * Kr[r], k[m].sum(axis=0), rtol=1e-10, atol=1e-10)
            np.testing.assert_allclose(w[r] * Vr[r], v[m].sum(axis=0), rtol=1e-10, atol=1e-10)
        if Br >= 1:
            assert len(pos) + int(w.sum()) == t + 1
        else:
            assert nr == 0 and rep.merge_slot == -1


def test_figure_caption_budgets(oracle):
    """Budgets printed with the paper's cache-operation figure: the steady-state occupancy
    they imply over the sequence lengths the caption names."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "kv_operation_budgets.txt"))
            if l.strip() and not l.startswith("#")]
    vals = {r[0]: int(r[1]) for r in rows}
    Br, Bc, Bp = vals["B_r"], vals["B_c"], vals["B_p"]
    rng = np.random.default_rng(1)
    q, k, v = heavy_hitter_stream(rng, vals["T_end"], 8, 1)
    u = oracle.Unit(8, 1, Bp, Bc, Br)
    for t in range(vals["T_end"]):
        u.decode_step(q[t], k[t], v[t])
        if t + 1 >= vals["T_start"]:
            np_, nc, nr, T = u.counts()
            assert (np_, nc, nr) == (Bp, Bc, Br)
            pos, _, _, _ = u.tokens()
            assert sorted(pos.tolist())[-Bp:] == list(range(t + 1 - Bp, t + 1))
            _, _, w = u.residual()
            assert len(pos) + int(w.sum()) == t + 1


@pytest.mark.parametrize("lam", [0.0, 0.98, 1.0])
def test_scores_brute_force(oracle, lam):
    """Eq. (score) unrolled: s_t^(T) = sum_tau lam^(T-tau) * mean_g a_hat_t^(tau), recomputed
    from the logged attention rows.  lam = 0 leaves the last row, lam = 1 the plain sum."""
    rng = np.random.default_rng(21)
    n, d, G = 70, 8, 2
    q, k, v = heavy_hitter_stream(rng, n, d, G)
    u = oracle.Unit(d, G, 5, 6, 2, lam=lam)
    rows = []
    for t in range(n):
        u.decode_step(q[t], k[t], v[t])
        a, ids = u.last_attention()
        rows.append({int(i): a[:, j].mean() for j, i in enumerate(ids) if i >= 0})
        pos, sc, _, _ = u.tokens()
        for p, s in zip(pos.tolist(), sc.tolist()):
            brute = sum((lam ** (t - tau)) * rows[tau][p] for tau in range(p, t + 1))
            assert abs(s - brute) <= 1e-5 * brute + 1e-30
            if lam == 0.0:
                assert s == np.float32(rows[t][p])


@pytest.mark.parametrize("alpha", [0.0, 1.0])
def test_pure_eviction_is_attention_over_retained_set(oracle, alpha):
    """B_r = 0 (Sec. 3.2: subsumes eviction): the output is plain attention restricted to
    the retained positions plus the new token, whatever alpha is."""
    rng = np.random.default_rng(33)
    n, d, G = 80, 8, 2
    q, k, v = heavy_hitter_stream(rng, n, d, G)
    u = oracle.Unit(d, G, 4, 5, 0, alpha=alpha)
    for t in range(n):
        pos_before = u.tokens()[0].tolist()
        o, _ = u.decode_step(q[t], k[t], v[t])
        keep = pos_before + [t]
        ref, _ = softmax_attention(q[t], k[keep], v[keep], 1 / np.sqrt(d))
        np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)


def test_alpha_zero_residual_is_unweighted_entry(oracle):
    """alpha = 0 (Sec. 3.5): a merged slot enters the softmax like one ordinary token whose
    key and value are the slot's means."""
    rng = np.random.default_rng(34)
    n, d = 60, 8
    q, k, v = heavy_hitter_stream(rng, n, d, 1)
    u = oracle.Unit(d, 1, 4, 5, 2, alpha=0.0)
    for t in range(n):
        pos, _, K, V = u.tokens()
        Kr, Vr, _ = u.residual()
        o, _ = u.decode_step(q[t], k[t], v[t])
        keys = np.concatenate([K, Kr, k[t][None]])
        vals = np.concatenate([V, Vr, v[t][None]])
        ref, _ = softmax_attention(q[t], keys, vals, 1 / np.sqrt(d))
        np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("budgets", [(6, 8, 2), (3, 4, 2), (1, 1, 1), (0, 5, 3), (5, 0, 2), (4, 6, 0), (16, 15, 1)])
@pytest.mark.parametrize("G", [1, 4])
def test_three_lists_equal_single_pool(oracle, budgets, G):
    """The literal three-list form and the single-pool form agree on every victim, every
    merge target, every output and the final state -- including under random shuffles of the
    pool's physical slots (ties are by position, not by slot)."""
    Bp, Bc, Br = budgets
    rng = np.random.default_rng(55 + G)
    n, d = 150, 16
    q, k, v = heavy_hitter_stream(rng, n, d, G)
    u = oracle.Unit(d, G, Bp, Bc, Br)
    pc = PoolCache(d, G, Bp, Bc, Br)
    for t in range(n):
        o1, rep = u.decode_step(q[t], k[t], v[t])
        if t % 7 == 3:
            pc.permute(rng)
        o2, vic, slot = pc.step(q[t], k[t], v[t])
        assert (rep.victim_pos, rep.merge_slot) == (vic, slot), t
        np.testing.assert_allclose(o1, o2, rtol=1e-11, atol=1e-13)
    pos, sc, K, V = u.tokens()
    order = np.argsort(pos)
    porder = np.argsort(pc.pos[: pc.n_live])
    np.testing.assert_array_equal(pos[order], pc.pos[: pc.n_live][porder])
    np.testing.assert_array_equal(sc[order], pc.s[: pc.n_live][porder])
    np.testing.assert_array_equal(K[order], pc.K[: pc.n_live][porder])
    Kr, Vr, w = u.residual()
    np.testing.assert_allclose(Kr, pc.Kr[: pc.n_res], rtol=1e-12)
    np.testing.assert_allclose(Vr, pc.Vr[: pc.n_res], rtol=1e-12)
    np.testing.assert_array_equal(w, pc.w[: pc.n_res])


@pytest.mark.parametrize("budgets", [(3, 4, 2), (0, 4, 1), (5, 0, 1), (2, 9, 0)])
def test_victim_is_brute_force_argmin(oracle, budgets):
    """Alg. 1 l.11 by brute force: from the state exported before the step and the logged
    attention row, recompute every updated score and take the minimum (score, position) over
    the tokens that are no longer among the B_p latest."""
    Bp, Bc, Br = budgets
    rng = np.random.default_rng(91)
    n, d, G, lam = 120, 8, 2, 0.98
    q, k, v = heavy_hitter_stream(rng, n, d, G)
    u = oracle.Unit(d, G, Bp, Bc, Br, lam=lam)
    n_checked = 0
    for t in range(n):
        pos_b, sc_b, _, _ = u.tokens()
        _, rep = u.decode_step(q[t], k[t], v[t])
        a, ids = u.last_attention()
        mean_a = {int(i): a[:, j].mean() for j, i in enumerate(ids) if i >= 0}
        upd = {int(p): np.float32(lam * float(s) + mean_a[int(p)]) for p, s in zip(pos_b, sc_b)}
        upd[t] = np.float32(mean_a[t])
        if len(upd) > Bp + Bc:
            cand = [(s, p) for p, s in upd.items() if p <= t - Bp]
            assert rep.victim_pos == min(cand)[1]
            n_checked += 1
        else:
            assert rep.victim_pos == -1
    assert n_checked > 50


def test_exact_tie_goes_to_lowest_position(oracle):
    """Two context tokens with bit-identical score histories: the lower position is evicted."""
    d = 4
    u = oracle.Unit(d, 1, Bp=1, Bc=2, Br=0, lam=0.0)   # lam = 0: score = last attention weight
    k_same = np.array([1.0, 0, 0, 0])
    k_hot = np.array([5.0, 0, 0, 0])
    q = np.array([[1.0, 0, 0, 0]])
    vv = np.ones(d)
    # positions 0,1 share a key (equal weights forever), later tokens are hotter
    u.decode_step(q, k_same, vv)
    u.decode_step(q, k_same, vv)
    u.decode_step(q, k_hot, vv)          # pos 2: proximity; context = {0, 1}
    _, rep = u.decode_step(q, k_hot, vv)  # pos 3: context {0,1,2} overflows
    assert rep.victim_pos == 0 and rep.victim_runner_pos == 1 and rep.victim_gap == 0.0
    _, rep = u.decode_step(q, k_hot, vv)
    assert rep.victim_pos == 1


def test_merge_target_is_max_raw_dot_product(oracle):
    """Eq. (hatr): raw dot product, not cosine -- a long slot key wins over a better aligned
    short one; equal dot products go to the lowest slot."""
    d = 4
    u = oracle.Unit(d, 1, Bp=1, Bc=1, Br=2, lam=0.0)
    q = np.array([[0.0, 0, 0, 1.0]])
    vv = np.zeros(d)
    toks = [np.array([10.0, 10.0, 0, -9]),   # pos 0 -> residual slot 0 (long, 45 degrees off)
            np.array([1.0, 0.0, 0, -9]),     # pos 1 -> residual slot 1 (short, aligned with pos 2)
            np.array([1.0, 0.0, 0, -8.5]),   # pos 2 -> merged: dot with slot0 = 86.5, slot1 = 77.5 (cosine prefers slot 1)
            np.array([0.0, 0.0, 0, 5.0]),
            np.array([0.0, 0.0, 0, 5.0])]
    reps = [u.decode_step(q, k, vv)[1] for k in toks]
    seq = [(r.victim_pos, r.merge_slot) for r in reps]
    assert seq[2] == (0, -2) and seq[3] == (1, -2)
    assert seq[4] == (2, 0)
    Kr, _, w = u.residual()
    np.testing.assert_allclose(Kr[0], (toks[0] + toks[2]) / 2)
    assert w.tolist()[0] == 2


@pytest.mark.parametrize("kind", ["identical", "equal_dot"])
def test_merge_tie_goes_to_lowest_slot(oracle, kind):
    """Eq. (hatr) with two slots that give the evicted token exactly the same dot product --
    bit-identical keys, or different keys whose products happen to agree: the lowest slot
    takes the token (small integers: every product and sum is exact)."""
    d = 4
    u = oracle.Unit(d, 1, Bp=1, Bc=1, Br=2, lam=0.0)
    q = np.array([[0.0, 0, 0, 1.0]])
    vv = np.arange(d, dtype=np.float64)
    second = [2.0, 0, 0, -40] if kind == "identical" else [0.0, 2.0, 0, -40]
    toks = [np.array([2.0, 0, 0, -40]),       # pos 0 -> residual slot 0
            np.array(second),                 # pos 1 -> residual slot 1
            np.array([1.0, 1.0, 0, -36]),     # pos 2: dot 1442 with slot 0 and with slot 1
            np.array([0.0, 0, 0, 20]), np.array([0.0, 0, 0, 20])]
    reps = [u.decode_step(q, k, vv * (i + 1))[1] for i, k in enumerate(toks)]
    seq = [(r.victim_pos, r.merge_slot) for r in reps]
    assert seq == [(-1, -1), (-1, -1), (0, -2), (1, -2), (2, 0)]
    assert reps[4].merge_runner_slot == 1 and reps[4].merge_gap == 0.0
    Kr, Vr, w = u.residual()
    assert w.tolist() == [2, 1]
    np.testing.assert_array_equal(Kr[0], (toks[0] + toks[2]) / 2)
    np.testing.assert_array_equal(Kr[1], toks[1])
    np.testing.assert_array_equal(Vr[0], (vv * 1 + vv * 3) / 2)


@pytest.mark.parametrize("Br", [2, 9, 40])
def test_planted_merge_ties_in_a_decode_stream(oracle, Br):
    """The planted-tie construction of tie_streams (pairs of slots front / back of the pool,
    identical keys or equal products, then tokens that tie between them) driven through the
    decode step: with lam = 1 and imported scores spaced far apart the victims come out in a
    known order, and each tie token must go to the lower slot of its pair."""
    from tie_streams import planted_prompt, tie_tokens
    d, Bp, Bc = 16, 10, 12     # B_p > number of steps: no decoded token leaves proximity
    rng = np.random.default_rng(40 + Br)
    ties, want = tie_tokens(Br, d)
    # prompt: the B_r slot fillers are evicted (they fill the slots); the tie tokens are kept
    # with the lowest scores, in order, so that decoding evicts them one per step
    K, V, s, n_ev, _ = planted_prompt(rng, d, Bp, Bc, Br, n_more=0)
    n_tie = len(want)
    assert 2 <= n_tie < Bp
    s[Br:Br + n_tie] = 10.0 * (1 + np.arange(n_tie))       # kept, evicted first later on
    s[Br + n_tie:] = 1000.0 + 10.0 * np.arange(len(s) - Br - n_tie)
    s[:Br] = 0.25
    u = oracle.Unit(d, 1, Bp, Bc + n_tie, Br, lam=1.0)
    res = u.prefill_compress(K, V, scores=s)
    assert np.flatnonzero(res.evicted).tolist() == list(range(Br)) and set(res.targets) == {-2}
    got = []
    for t in range(n_tie):
        q = rng.normal(size=(1, d))
        _, rep = u.decode_step(q, rng.normal(size=d), rng.normal(size=d))
        assert rep.victim_pos == Br + t
        assert rep.merge_gap == 0.0
        got.append(rep.merge_slot)
    assert got == want


def test_cosine_form_prefers_the_aligned_slot(oracle):
    """The cosine form of Eq. (hatr) (commented out beside it in the paper's source): on the
    same stream as above the better aligned short slot wins, and every merge target of a
    random stream is the brute-force argmax of k_r.k_t / (|k_r||k_t|) over the merged keys as
    they stood before the step."""
    d = 4
    u = oracle.Unit(d, 1, Bp=1, Bc=1, Br=2, lam=0.0, cosine=True)
    q = np.array([[0.0, 0, 0, 1.0]])
    vv = np.zeros(d)
    toks = [np.array([10.0, 10.0, 0, -9]), np.array([1.0, 0.0, 0, -9]),
            np.array([1.0, 0.0, 0, -8.5]), np.array([0.0, 0.0, 0, 5.0]),
            np.array([0.0, 0.0, 0, 5.0])]
    reps = [u.decode_step(q, k, vv)[1] for k in toks]
    assert (reps[4].victim_pos, reps[4].merge_slot) == (2, 1)
    Kr, _, w = u.residual()
    np.testing.assert_allclose(Kr[1], (toks[1] + toks[2]) / 2)
    assert w.tolist() == [1, 2]

    rng = np.random.default_rng(77)
    n, d, G = 120, 16, 2
    qs, ks, vs = heavy_hitter_stream(rng, n, d, G)
    ks = ks * rng.uniform(0.2, 5.0, size=(n, 1))  # very different key lengths
    u = oracle.Unit(d, G, Bp=5, Bc=9, Br=4, cosine=True)
    ud = oracle.Unit(d, G, Bp=5, Bc=9, Br=4)
    merges = differ = 0
    for t in range(n):
        pos, _, Kt, _ = u.tokens()
        Kr, _, _ = u.residual()
        _, rep = u.decode_step(qs[t], ks[t], vs[t])
        _, repd = ud.decode_step(qs[t], ks[t], vs[t])
        if rep.merge_slot >= 0:
            kv = Kt[list(pos).index(rep.victim_pos)]
            cos = (Kr @ kv) / (np.linalg.norm(Kr, axis=1) * np.linalg.norm(kv))
            assert rep.merge_slot == int(np.argmax(cos.astype(np.float32)))
            merges += 1
        differ += int(rep.merge_slot != repd.merge_slot)
    assert merges > 80 and differ > 0  # and the two forms do part ways on such keys


def test_hint_protocol(oracle):
    """A hinted choice is taken only inside the tolerance; otherwise the oracle keeps its own
    and flags the mismatch."""
    rng = np.random.default_rng(77)
    n, d = 40, 8
    q, k, v = heavy_hitter_stream(rng, n, d, 1)
    u = oracle.Unit(d, 1, 3, 4, 2)
    free = oracle.Unit(d, 1, 3, 4, 2)
    for t in range(n):
        _, rf = free.decode_step(q[t], k[t], v[t])
        if rf.victim_pos >= 0 and rf.victim_runner_pos >= 0 and t == 30:
            # a far-off runner-up must be refused ...
            _, r = u.decode_step(q[t], k[t], v[t], hint_victim=rf.victim_runner_pos, tol=1e-9)
            assert r.victim_mismatch == 1 and r.victim_pos == rf.victim_pos
        elif rf.victim_pos >= 0 and rf.victim_runner_pos >= 0 and t == 35:
            # ... and accepted once the tolerance covers the gap
            _, r = u.decode_step(q[t], k[t], v[t], hint_victim=rf.victim_runner_pos,
                                 tol=rf.victim_gap * 1.01)
            assert r.victim_near_tie == 1 and r.victim_pos == rf.victim_runner_pos
            assert r.victim_own_pos == rf.victim_pos
            break
        else:
            _, r = u.decode_step(q[t], k[t], v[t], hint_victim=rf.victim_pos,
                                 hint_slot=rf.merge_slot, tol=1e-4)
            assert (r.victim_near_tie, r.victim_mismatch, r.merge_near_tie, r.merge_mismatch) == (0, 0, 0, 0)
            assert (r.victim_pos, r.merge_slot) == (rf.victim_pos, rf.merge_slot)


def test_batch_entry_matches_single(oracle):
    rng = np.random.default_rng(8)
    n_units, n, d, G = 5, 30, 8, 2
    streams = [heavy_hitter_stream(rng, n, d, G) for _ in range(n_units)]
    a = [oracle.Unit(d, G, 3, 4, 1) for _ in range(n_units)]
    b = [oracle.Unit(d, G, 3, 4, 1) for _ in range(n_units)]
    for t in range(n):
        q = np.stack([s[0][t] for s in streams])
        k = np.stack([s[1][t] for s in streams])
        v = np.stack([s[2][t] for s in streams])
        out, threads = oracle.decode_step_batch(a, q, k, v)
        assert threads >= 1
        for i in range(n_units):
            o, _ = b[i].decode_step(q[i], k[i], v[i])
            np.testing.assert_array_equal(out[i], o)


def test_budget_split_golden(oracle):
    """App. C.2 ratios (tail 0.5, dense 0.02) on the budgets of the five workloads."""
    for line in open(os.path.join(GOLDEN, "budget_split.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        B, bp, bc, br = (int(x) for x in line.split())
        assert oracle.split_budget(B) == (bp, bc, br)
        assert bp + bc + br == B
    assert oracle.split_budget(100, 0.5, 0.0) == (50, 50, 0)


def test_budget_split_holds_the_two_ratios(oracle):
    """App. C.2 fixes two ratios: B_p / B (0.5 recommended) and B_r / (B - B_p) (0.02).  However
    the helper rounds, an integer split can be held to them: B_p within one slot of 0.5 B,
    B_r within half a slot of 0.02 (B - B_p) or at its floor of one slot, B_c the remainder."""
    for B in list(range(1, 3000)) + list(range(3000, 60001, 37)) + [60000]:
        bp, bc, br = oracle.split_budget(B)
        assert bp + bc + br == B and min(bp, bc, br) >= 0 and bp + bc >= 1
        assert abs(bp - 0.5 * B) < 1.0
        assert abs(br - 0.02 * (B - bp)) <= 0.5 or br == 1 or (br == 0 and B == 1)
    for tail, dense in [(0.3, 0.05), (0.7, 0.1), (0.5, 0.2), (0.1, 0.01)]:
        for B in (64, 205, 819, 2700, 10800, 54000):
            bp, bc, br = oracle.split_budget(B, tail, dense)
            assert bp + bc + br == B and abs(bp - tail * B) < 1.0
            assert abs(br - dense * (B - bp)) <= 0.5 or br == 1
