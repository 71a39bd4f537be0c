"""GPU parity of the full-history prompt scores (every prompt query scores every earlier key)
against the oracle's prompt pass with the window taken as the whole prompt, against the
definition written out with a library softmax, and end to end into the compression."""
import numpy as np
import pytest
import torch

import workloads as wl
from harness import GpuCache, ParityStats, SCORE_RTOL, f64, oracle_unit_for, prefill_check

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import binding
    return binding


def full_scores(zb, cache, K, Q, lse=None):
    T = K.shape[2]
    w = cache.w
    scores = torch.full((w.batch, w.n_kv_heads, T), float("nan"), dtype=torch.float32, device="cuda")
    ws = None
    if lse is None:
        ws = torch.empty(zb.zsm_prefill_scores_full_workspace_bytes(cache.h, T), dtype=torch.uint8,
                         device="cuda")
    zb.zsm_prefill_scores_full(cache.h, K, Q, T, scores, ws, lse)
    torch.cuda.synchronize()
    return scores, ws


def oracle_scores(oracle, cache, K, V, Q, b, h):
    G = cache.w.group
    unit = oracle_unit_for(oracle, cache, 0, h)
    return unit.prefill_compress(f64(K[b, h]), f64(V[b, h]), Qw=f64(Q[b, h * G:(h + 1) * G])).scores


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("head_dim,group", [(64, 1), (128, 1), (128, 4), (64, 2)])
def test_full_scores_match_the_oracle(zb, oracle, dtype, head_dim, group):
    """Several 64-row blocks with a ragged last one, every kernel variant."""
    T = 333
    w = wl.Workload("full", 1, 2, 2 * group, 2, head_dim, dtype, T, 0, T, None, 31)
    cache = GpuCache(zb, w, [[8, 12]], [[20, 30]], [[2, 3]])
    try:
        K, V, Q = wl.prompt(w, 0)
        s_gpu, _ = full_scores(zb, cache, K.cuda(), Q.cuda())
        s_gpu = s_gpu.cpu().numpy().astype(np.float64)
        assert np.isfinite(s_gpu).all()
        for b in range(w.batch):
            for h in range(w.n_kv_heads):
                ref = oracle_scores(oracle, cache, K, V, Q, b, h).astype(np.float64)
                rel = np.abs(s_gpu[b, h] - ref) / np.maximum(np.abs(ref), 1e-30)
                assert rel.max() <= SCORE_RTOL, f"unit {(b, h)}: relative error {rel.max():.3e}"
    finally:
        cache.close()


@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 128, 200])
@pytest.mark.parametrize("lam", [0.98, 1.0, 0.0])
def test_full_scores_against_the_definition(zb, T, lam):
    """Block edges, the shortest prompts and the ends of the decay range, against the column
    sums of a causal softmax matrix computed with torch in fp64; also with the row statistics
    handed in instead of computed."""
    w = wl.Workload("fulldef", 1, 1, 4, 2, 128, "f16", T, 0, T, None, 32)
    cache = GpuCache(zb, w, [[4, 4]], [[4, 4]], [[1, 1]], lam=lam)
    try:
        K, V, Q = wl.prompt(w, 0)
        s_gpu, ws = full_scores(zb, cache, K.cuda(), Q.cuda())
        G = w.group
        Kd, Qd = K.double(), Q.double()
        logits = torch.einsum("bhgqd,bhkd->bhgqk", Qd.view(1, 2, G, T, 128), Kd) / np.sqrt(128.0)
        mask = torch.tril(torch.ones(T, T, dtype=torch.bool))
        logits = logits.masked_fill(~mask, float("-inf"))
        A = torch.softmax(logits, dim=-1)                       # [b, h, g, query, key]
        decay = torch.tensor([1.0 if q == T - 1 else float(lam) ** (T - 1 - q) for q in range(T)],
                             dtype=torch.float64)
        ref = (A * decay.view(1, 1, 1, T, 1)).sum(dim=3).mean(dim=2)  # [b, h, key]
        got = s_gpu.cpu().double()
        err = (got - ref).abs() / ref.abs().clamp_min(1e-30)
        nz = ref > 0
        assert err[nz].max().item() <= SCORE_RTOL if nz.any() else True
        assert (got[~nz] == 0).all()
        # the same with the log-sum-exp of each row supplied by the caller
        lse = torch.logsumexp(logits, dim=-1).view(1, 2 * G, T).float().cuda().contiguous()
        s2, _ = full_scores(zb, cache, K.cuda(), Q.cuda(), lse=lse)
        err2 = (s2.cpu().double() - ref).abs() / ref.abs().clamp_min(1e-30)
        assert err2[nz].max().item() <= SCORE_RTOL if nz.any() else True
    finally:
        cache.close()


@pytest.mark.parametrize("dtype,head_dim,group,T", [("bf16", 128, 4, 8192 + 77), ("f16", 64, 2, 8192 + 130)])
def test_full_scores_at_long_prompts(zb, oracle, dtype, head_dim, group, T):
    """A prompt of more than 64 key blocks with grouped heads: every CTA walks hundreds of
    (tile, head) items, so the tile ring, the exponent-offset ring and the accumulator phases
    wrap many times.  The oracle's full-history pass is quadratic, so one sampled head per
    sequence is recomputed; the rest are held to what holds for any input (finite, positive,
    and the column sums of a softmax matrix add up to the sum of the decay weights)."""
    w = wl.Workload("fulllong", 1, 2, 3 * group, 3, head_dim, dtype, T, 0, T, None, 38)
    cache = GpuCache(zb, w, [[8] * 3], [[20] * 3], [[2] * 3])
    try:
        K, V, Q = wl.prompt(w, 0)
        s_gpu, _ = full_scores(zb, cache, K.cuda(), Q.cuda())
        assert cache.status() == 0
        s_gpu = s_gpu.cpu().numpy().astype(np.float64)
        assert np.isfinite(s_gpu).all() and (s_gpu > 0).all()
        lam = float(np.float32(cache.lam))
        total = sum(lam ** (T - 1 - q) for q in range(T))        # each softmax row sums to one
        np.testing.assert_allclose(s_gpu.sum(axis=-1), total, rtol=1e-5)
        for b, h in [(0, 1), (1, 2)]:
            ref = oracle_scores(oracle, cache, K, V, Q, b, h).astype(np.float64)
            rel = np.abs(s_gpu[b, h] - ref) / np.maximum(np.abs(ref), 1e-30)
            assert rel.max() <= SCORE_RTOL, f"unit {(b, h)}: relative error {rel.max():.3e}"
    finally:
        cache.close()


def test_full_scores_feed_the_compression(zb, oracle):
    """Scores from the full-history pass, handed to the compression as precomputed scores, give
    the oracle's selection, merge chain and state for a window equal to the prompt."""
    T = 500
    w = wl.Workload("fullpp", 1, 1, 4, 2, 128, "bf16", T, 0, T, None, 33)
    cache = GpuCache(zb, w, [[16, 24]], [[40, 56]], [[3, 6]])
    stats = ParityStats()
    try:
        K, V, Q = wl.prompt(w, 0)
        s_gpu, _ = full_scores(zb, cache, K.cuda(), Q.cuda())
        dbg = cache.prefill(0, K.cuda(), V.cuda(), None, s_gpu)
        for h in range(w.n_kv_heads):
            prefill_check(oracle, cache, 0, 0, h, K, V, Q, dbg, stats,
                          scores_given=s_gpu[0, h].cpu().numpy(), tag=f"unit {h}")
        assert cache.status() == 0 and stats.merges > 500
    finally:
        cache.close()


def test_full_scores_argument_errors(zb):
    w = wl.Workload("fullerr", 1, 1, 2, 2, 64, "f32", 32, 0, 32, None, 34)
    cache = GpuCache(zb, w, [[4, 4]], [[4, 4]], [[1, 1]])
    try:
        K, V, Q = (t.cuda() for t in wl.prompt(w, 0))
        s = torch.empty(1, 2, 32, dtype=torch.float32, device="cuda")
        ws = torch.empty(zb.zsm_prefill_scores_full_workspace_bytes(cache.h, 32), dtype=torch.uint8,
                         device="cuda")
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_prefill_scores_full(cache.h, K, Q, 32, s, ws)
        assert e.value.status == zb.ZSM_ERR_UNSUPPORTED  # fp32 storage
    finally:
        cache.close()
    w = w.replace(dtype="f16")
    cache = GpuCache(zb, w, [[4, 4]], [[4, 4]], [[1, 1]])
    try:
        K, V, Q = (t.cuda() for t in wl.prompt(w, 0))
        s = torch.empty(1, 2, 32, dtype=torch.float32, device="cuda")
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_prefill_scores_full(cache.h, K, Q, 32, s, None)
        assert e.value.status == zb.ZSM_ERR_INVALID_ARG  # no workspace and no row statistics
        small = torch.empty(128, dtype=torch.uint8, device="cuda")
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_prefill_scores_full(cache.h, K, Q, 32, s, small)
        assert e.value.status == zb.ZSM_ERR_BUFFER_TOO_SMALL
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_prefill_scores_full(cache.h, K, Q, 0, s, small)
        assert e.value.status == zb.ZSM_ERR_INVALID_ARG
    finally:
        cache.close()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("head_dim,group,T", [(128, 1, 333), (128, 4, 700), (64, 2, 129), (64, 1, 1), (128, 2, 128)])
def test_prefill_attention_output_lse_and_scores(zb, oracle, dtype, head_dim, group, T):
    """zsm_prefill_attention: the causal attention output against torch's SDPA in fp64, the rows'
    log-sum-exp against torch.logsumexp, and the scores it leaves behind against the oracle's
    full-history prompt pass (one sampled head per sequence when the prompt is long)."""
    w = wl.Workload("attn", 1, 2, 2 * group, 2, head_dim, dtype, T, 0, T, None, 41)
    cache = GpuCache(zb, w, [[4, 4]], [[6, 6]], [[1, 1]])
    try:
        K, V, Q = wl.prompt(w, 0)
        dev = "cuda"
        out = torch.full((w.batch, w.n_q_heads, T, head_dim), float("nan"), dtype=w.torch_dtype, device=dev)
        lse = torch.full((w.batch, w.n_q_heads, T), float("nan"), dtype=torch.float32, device=dev)
        scores = torch.full((w.batch, w.n_kv_heads, T), float("nan"), dtype=torch.float32, device=dev)
        zb.zsm_prefill_attention(cache.h, K.cuda(), V.cuda(), Q.cuda(), T, out, lse, scores)
        torch.cuda.synchronize()
        assert cache.status() == 0
        Kd = K.double().repeat_interleave(group, dim=1)
        Vd = V.double().repeat_interleave(group, dim=1)
        Qd = Q.double()
        ref = torch.nn.functional.scaled_dot_product_attention(Qd, Kd, Vd, is_causal=True)
        torch.testing.assert_close(out.cpu().double(), ref, atol=2e-3, rtol=1e-2)
        logits = torch.einsum("bhqd,bhkd->bhqk", Qd, Kd) / np.sqrt(float(head_dim))
        mask = torch.tril(torch.ones(T, T, dtype=torch.bool))
        ref_lse = torch.logsumexp(logits.masked_fill(~mask, float("-inf")), dim=-1)
        torch.testing.assert_close(lse.cpu().double(), ref_lse, atol=1e-4, rtol=1e-5)
        s_gpu = scores.cpu().numpy().astype(np.float64)
        for b, h in [(0, 0), (1, 1)]:
            sref = oracle_scores(oracle, cache, K, V, Q, b, h).astype(np.float64)
            rel = np.abs(s_gpu[b, h] - sref) / np.maximum(np.abs(sref), 1e-30)
            assert rel.max() <= SCORE_RTOL, f"unit {(b, h)}: relative error {rel.max():.3e}"
        # without `scores` only the output and the row statistics are produced
        out2 = torch.empty_like(out)
        lse2 = torch.empty_like(lse)
        zb.zsm_prefill_attention(cache.h, K.cuda(), V.cuda(), Q.cuda(), T, out2, lse2)
        torch.cuda.synchronize()
        assert torch.equal(out2, out) and torch.equal(lse2, lse)
    finally:
        cache.close()


def test_prefill_attention_long_prompt(zb):
    """Many key tiles per query block (the S accumulators, the weight tile, both tile rings and
    every barrier phase wrap dozens of times), grouped heads; output against SDPA in fp64 on a
    sample of heads, row sums of the weights through the log-sum-exp."""
    T, d, G = 4096 + 57, 128, 4
    w = wl.Workload("attnlong", 1, 1, 2 * G, 2, d, "bf16", T, 0, T, None, 42)
    cache = GpuCache(zb, w, [[4, 4]], [[6, 6]], [[1, 1]])
    try:
        K, V, Q = wl.prompt(w, 0)
        out = torch.empty(1, 2 * G, T, d, dtype=torch.bfloat16, device="cuda")
        lse = torch.empty(1, 2 * G, T, dtype=torch.float32, device="cuda")
        zb.zsm_prefill_attention(cache.h, K.cuda(), V.cuda(), Q.cuda(), T, out, lse)
        torch.cuda.synchronize()
        assert cache.status() == 0
        for hq in (0, 5):
            hk = hq // G
            ref = torch.nn.functional.scaled_dot_product_attention(
                Q[:, hq:hq + 1].double(), K[:, hk:hk + 1].double(), V[:, hk:hk + 1].double(), is_causal=True)
            torch.testing.assert_close(out[:, hq:hq + 1].cpu().double(), ref, atol=2e-3, rtol=1e-2)
            logits = (Q[0, hq].double() @ K[0, hk].double().T) / np.sqrt(float(d))
            mask = torch.tril(torch.ones(T, T, dtype=torch.bool))
            ref_lse = torch.logsumexp(logits.masked_fill(~mask, float("-inf")), dim=-1)
            torch.testing.assert_close(lse[0, hq].cpu().double(), ref_lse, atol=1e-4, rtol=1e-5)
    finally:
        cache.close()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_prefill_attention_rising_maximum(zb, dtype):
    """Logits that keep growing with the key position, by about 18 in the log2 domain per key
    tile, for the odd query rows only: the reference maximum of those rows moves at every tile, so
    their rows of the output accumulator are rescaled in tensor memory again and again, while the
    even rows of the same warps (flat logits) keep theirs.  Output against SDPA in fp64, log-sum-exp
    against torch.logsumexp."""
    T, d, G = 700, 128, 2
    w = wl.Workload("attnrise", 1, 1, 2 * G, 2, d, dtype, T, 0, T, None, 44)
    cache = GpuCache(zb, w, [[4, 4]], [[6, 6]], [[1, 1]])
    try:
        K, V, Q = wl.prompt(w, 0)
        ramp = torch.arange(T, dtype=torch.float32) * 0.1      # logit gain per key position
        K = K.float() * 0.05
        K[..., 0] = ramp                                        # keys grow along the first axis
        Q = Q.float() * 0.05
        Q[..., 0] = 0.0
        Q[:, :, 1::2, 0] = float(np.sqrt(d))                    # odd rows: logit = 0.1 * position
        K, Q = K.to(w.torch_dtype), Q.to(w.torch_dtype)
        out = torch.full((1, 2 * G, T, d), float("nan"), dtype=w.torch_dtype, device="cuda")
        lse = torch.full((1, 2 * G, T), float("nan"), dtype=torch.float32, device="cuda")
        zb.zsm_prefill_attention(cache.h, K.cuda(), V.cuda(), Q.cuda(), T, out, lse)
        torch.cuda.synchronize()
        assert cache.status() == 0
        Kd = K.double().repeat_interleave(G, dim=1)
        Vd = V.double().repeat_interleave(G, dim=1)
        Qd = Q.double()
        ref = torch.nn.functional.scaled_dot_product_attention(Qd, Kd, Vd, is_causal=True)
        torch.testing.assert_close(out.cpu().double(), ref, atol=2e-3, rtol=1e-2)
        logits = torch.einsum("bhqd,bhkd->bhqk", Qd, Kd) / np.sqrt(float(d))
        mask = torch.tril(torch.ones(T, T, dtype=torch.bool))
        ref_lse = torch.logsumexp(logits.masked_fill(~mask, float("-inf")), dim=-1)
        # the rise over the prompt is what the test is about: 0.1 * 699 nats on the odd rows
        assert float(ref_lse[0, 0, T - 1]) > 60.0 and abs(float(ref_lse[0, 0, T - 2])) < 10.0
        torch.testing.assert_close(lse.cpu().double(), ref_lse, atol=1e-4, rtol=1e-5)
    finally:
        cache.close()


def test_prefill_attention_argument_errors(zb):
    w = wl.Workload("attnerr", 1, 1, 2, 2, 64, "f32", 32, 0, 32, None, 43)
    cache = GpuCache(zb, w, [[4, 4]], [[4, 4]], [[1, 1]])
    try:
        K, V, Q = (t.cuda() for t in wl.prompt(w, 0))
        out = torch.empty_like(Q)
        lse = torch.empty(1, 2, 32, dtype=torch.float32, device="cuda")
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_prefill_attention(cache.h, K, V, Q, 32, out, lse)
        assert e.value.status == zb.ZSM_ERR_UNSUPPORTED  # fp32 storage
        with pytest.raises(ValueError):
            zb.zsm_prefill_attention(cache.h, K, V, Q, 64, out, lse)  # tensors shorter than T says
    finally:
        cache.close()
