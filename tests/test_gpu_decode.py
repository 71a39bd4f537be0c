"""GPU parity of the fused decode step against the oracle, element by element, through
the C ABI.  Small and medium shapes that span several tiles and ragged tails; the
degenerate budgets the method has; both launch shapes (all layers / one layer)."""
import numpy as np
import pytest
import torch

import workloads as wl
from harness import (GpuCache, ParityStats, f64, oracle_step_check, oracle_unit_for, split_budgets,
                     state_check)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import binding
    return binding


def run_decode(zb, oracle, w, bp, bc, br, steps, layer_mode=-1, check_state_every=25, alpha=1.0,
               lam=0.98, units=None, **tune):
    cache = GpuCache(zb, w, bp, bc, br, lam=lam, alpha=alpha, **tune)
    stats = ParityStats()
    try:
        if units is None:
            units = [(l, b, h) for l in range(w.n_layers) for b in range(w.batch)
                     for h in range(w.n_kv_heads)]
        orc = {u: oracle_unit_for(oracle, cache, u[0], u[2]) for u in units}
        G = w.group
        for step in range(steps):
            q, k, v = wl.decode_inputs(w, step)
            out, vic, slot = cache.decode(q.cuda(), k.cuda(), v.cuda(), layer=layer_mode)
            out_h, vic_h, slot_h = f64(out), vic.cpu().numpy(), slot.cpu().numpy()
            q64, k64, v64 = f64(q), f64(k), f64(v)
            for (l, b, h), unit in orc.items():
                oracle_step_check(unit, q64[l, b, h * G:(h + 1) * G], k64[l, b, h], v64[l, b, h],
                                  out_h[l, b, h * G:(h + 1) * G], vic_h[l, b, h], slot_h[l, b, h],
                                  w.dtype, stats, tag=f"step {step} unit {(l, b, h)}")
            if (step + 1) % check_state_every == 0 or step == steps - 1:
                for (l, b, h), unit in orc.items():
                    state_check(unit, cache.export(l, b, h), stats, tag=f"step {step} unit {(l, b, h)}")
        assert cache.status() == 0
    finally:
        cache.close()
    assert stats.exact_tie_breaches == 0
    return stats


SMALL = wl.Workload("small", 2, 2, 2, 2, 64, "f32", 0, 0, 0, None, 11)


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("head_dim", [64, 128])
@pytest.mark.parametrize("group", [1, 4])
@pytest.mark.parametrize("split", [0, 1])
def test_decode_from_empty_all_kernel_variants(zb, oracle, dtype, head_dim, group, split):
    """Every (dtype, head_dim, group) kernel, in the split form (a cluster of CTAs per unit: the
    library's choice for so few units) and with one CTA per unit: fill, first evictions,
    residual fill, merges."""
    w = SMALL.replace(dtype=dtype, head_dim=head_dim, n_q_heads=2 * group)
    bp = np.array([[6, 9], [4, 20]])
    bc = np.array([[7, 30], [5, 11]])
    br = np.array([[2, 3], [1, 5]])
    stats = run_decode(zb, oracle, w, bp, bc, br, steps=90, tune_split=split)
    assert stats.selections > 200 and stats.merges > 150


@pytest.mark.parametrize("budgets", [(0, 5, 3), (5, 0, 2), (4, 6, 0), (1, 1, 1), (0, 1, 0), (1, 0, 1)])
@pytest.mark.parametrize("split", [0, 1])
def test_degenerate_budgets(zb, oracle, budgets, split):
    """B_p = 0 (the new token competes at once), B_c = 0 (whatever leaves proximity is evicted),
    B_r = 0 (pure eviction) and the smallest caches -- in the split form most CTAs of a cluster
    then have no slot at all."""
    w = SMALL.replace(dtype="f16", head_dim=128, n_layers=1)
    bp, bc, br = (np.full((1, 2), x) for x in budgets)
    run_decode(zb, oracle, w, bp, bc, br, steps=40, check_state_every=5, tune_split=split)


@pytest.mark.parametrize("alpha,lam", [(0.0, 0.98), (0.5, 0.5), (1.0, 0.0), (1.0, 1.0)])
def test_alpha_and_lambda_range(zb, oracle, alpha, lam):
    w = SMALL.replace(dtype="f16", head_dim=128, n_layers=1)
    run_decode(zb, oracle, w, np.full((1, 2), 5), np.full((1, 2), 6), np.full((1, 2), 2), steps=50,
               alpha=alpha, lam=lam)


@pytest.mark.parametrize("split", [0, 1])
@pytest.mark.parametrize("layer_mode", [-1, "each"])
def test_multi_tile_ragged_units(zb, oracle, layer_mode, split):
    """Slot pools that span several 16 KiB tiles with a ragged last tile, ragged per-head
    budgets, residual pools larger than one tile row group; both launch shapes."""
    w = wl.Workload("ragged", 2, 2, 8, 4, 128, "f16", 0, 0, 0, None, 12)
    rs = np.random.RandomState(5)
    tot = rs.randint(70, 260, size=(2, 4))
    bp, bc, br = split_budgets(zb, tot)
    br[0, 1], br[1, 2] = 37, 0
    stats = run_decode(zb, oracle, w, bp, bc, br, steps=300, layer_mode=layer_mode,
                       check_state_every=100, tune_split=split)
    assert stats.selections > 1000


def test_budget_at_least_context_is_full_attention(zb):
    """Invariant: while nothing is evicted the output is plain softmax attention over the
    whole history (checked against torch SDPA in fp64 on the CPU, not against the oracle)."""
    w = wl.Workload("full", 1, 2, 4, 2, 128, "f16", 0, 0, 0, None, 13)
    steps = 150
    cache = GpuCache(zb, w, np.full((1, 2), 40), np.full((1, 2), steps), np.full((1, 2), 3))
    try:
        qs, ks, vs = [], [], []
        for step in range(steps):
            q, k, v = wl.decode_inputs(w, step)
            out, vic, _ = cache.decode(q.cuda(), k.cuda(), v.cuda())
            qs.append(q[0]), ks.append(k[0]), vs.append(v[0])
            K = torch.stack(ks, dim=2).double().repeat_interleave(w.group, dim=1)   # [b,Hq,t,d]
            V = torch.stack(vs, dim=2).double().repeat_interleave(w.group, dim=1)
            ref = torch.nn.functional.scaled_dot_product_attention(q[0].double()[:, :, None, :], K, V)
            torch.testing.assert_close(out[0].cpu().double(), ref[:, :, 0, :], atol=2e-3, rtol=1e-2)
            assert (vic.cpu() == -1).all()
        assert cache.status() == 0
    finally:
        cache.close()


def test_decode_from_imported_large_state(zb, oracle):
    """A unit larger than one (score, pos) tile (2048 entries) and a residual pool of 60
    slots: state built by the oracle's prompt pass, imported through the C ABI, then decoded
    on both sides."""
    w = wl.Workload("large", 1, 1, 2, 1, 128, "bf16", 0, 0, 0, None, 15)
    bp, bc, br = 1100, 1250, 60
    T = 3000
    g = torch.Generator().manual_seed(3)
    K = torch.randn(T, 128, generator=g).to(torch.bfloat16)
    V = torch.randn(T, 128, generator=g).to(torch.bfloat16)
    scores = torch.rand(T, generator=g).numpy().astype(np.float32) + 1e-3
    cache = GpuCache(zb, w, [[bp]], [[bc]], [[br]])
    stats = ParityStats()
    try:
        unit = oracle_unit_for(oracle, cache, 0, 0)
        unit.prefill_compress(f64(K), f64(V), scores=scores)
        pos, sc, Kt, Vt = unit.tokens()
        Kr, Vr, wr = unit.residual()
        state = dict(K=Kt, V=Vt, score=sc, pos=pos, Kr=Kr, Vr=Vr, w=wr, n_live=len(pos),
                     n_res=len(wr), T=T)
        zb.zsm_cache_import_unit(cache.h, 0, 0, 0, 128, state)
        state_check(unit, cache.export(0, 0, 0), stats, tag="after import")
        for step in range(60):
            q, k, v = wl.decode_inputs(w, step)
            out, vic, slot = cache.decode(q.cuda(), k.cuda(), v.cuda())
            oracle_step_check(unit, f64(q)[0, 0], f64(k)[0, 0, 0], f64(v)[0, 0, 0], f64(out)[0, 0],
                              int(vic.cpu()[0, 0, 0]), int(slot.cpu()[0, 0, 0]), w.dtype, stats,
                              tag=f"step {step}")
        state_check(unit, cache.export(0, 0, 0), stats, tag="end")
        assert cache.status() == 0 and stats.merges == 60
    finally:
        cache.close()


def test_host_buffer_entry_point_matches_device_entry_point(zb):
    """zsm_decode_step_host = copies in, the same kernel, copy out."""
    w = wl.Workload("host", 2, 2, 4, 2, 128, "f16", 0, 0, 0, None, 16)
    mk = lambda: GpuCache(zb, w, np.full((2, 2), 8), np.full((2, 2), 9), np.full((2, 2), 2))
    a, b = mk(), mk()
    try:
        staging = torch.empty(zb.zsm_decode_staging_bytes(b.h, -1), dtype=torch.uint8, device="cuda")
        for step in range(40):
            q, k, v = wl.decode_inputs(w, step)
            out, _, _ = a.decode(q.cuda(), k.cuda(), v.cuda())
            qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
            oh = torch.empty_like(qh).pin_memory()
            zb.zsm_decode_step_host(b.h, -1, qh, kh, vh, oh, staging)
            assert torch.equal(out.cpu(), oh)
        assert a.status() == 0 and b.status() == 0
    finally:
        a.close(), b.close()


def test_pipelined_host_buffer_steps_match_device_entry_point(zb):
    """zsm_decode_step_host_async over two staging halves: same outputs, step for step, as the
    device entry point, with two steps in flight at a time."""
    w = wl.Workload("hostpipe", 2, 2, 4, 2, 128, "bf16", 0, 0, 0, None, 39)
    mk = lambda: GpuCache(zb, w, np.full((2, 2), 8), np.full((2, 2), 9), np.full((2, 2), 2))
    a, b = mk(), mk()
    try:
        q_off, k_off, v_off, in_bytes, out_bytes = zb.zsm_decode_host_layout(b.h, -1)
        half = in_bytes + (out_bytes + 255) // 256 * 256
        staging = torch.empty(2 * half, dtype=torch.uint8, device="cuda")
        ins = [torch.zeros(in_bytes, dtype=torch.uint8).pin_memory() for _ in range(2)]
        outs = [torch.empty(w.n_layers, w.batch, w.n_q_heads, w.head_dim,
                            dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_decode_step_host_wait(b.h, 0)
        assert e.value.status == zb.ZSM_ERR_STATE
        steps, ref = 41, []
        for step in range(steps):
            q, k, v = wl.decode_inputs(w, step)
            out, _, _ = a.decode(q.cuda(), k.cuda(), v.cuda())
            ref.append(out.cpu().clone())
        def pack(dst, q, k, v):
            for off, t in ((q_off, q), (k_off, k), (v_off, v)):
                raw = t.contiguous().view(torch.uint8).reshape(-1)
                dst[off:off + raw.numel()] = raw
        got = [None] * steps
        for step in range(steps + 1):
            slot = step & 1
            if step >= 2 or step == steps:
                pass
            if step >= 2:                       # the slot's previous step must be done before reuse
                zb.zsm_decode_step_host_wait(b.h, slot)
                got[step - 2] = outs[slot].clone()
            if step < steps:
                pack(ins[slot], *wl.decode_inputs(w, step))
                zb.zsm_decode_step_host_async(b.h, -1, ins[slot], outs[slot], staging, slot)
        zb.zsm_decode_step_host_wait(b.h, (steps - 1) & 1)
        got[steps - 1] = outs[(steps - 1) & 1].clone()
        for step in range(steps):
            assert torch.equal(got[step], ref[step]), f"step {step}"
        assert a.status() == 0 and b.status() == 0
    finally:
        a.close(), b.close()


def test_runs_are_bitwise_reproducible(zb):
    w = wl.Workload("repro", 2, 2, 8, 2, 128, "bf16", 0, 0, 0, None, 17)
    outs = []
    for _ in range(2):
        c = GpuCache(zb, w, np.full((2, 2), 20), np.full((2, 2), 90), np.full((2, 2), 4))
        try:
            acc = []
            for step in range(150):
                q, k, v = wl.decode_inputs(w, step)
                out, vic, slot = c.decode(q.cuda(), k.cuda(), v.cuda())
                acc.append((out.clone(), vic.clone(), slot.clone()))
            outs.append(acc)
        finally:
            c.close()
    for (o1, v1, s1), (o2, v2, s2) in zip(*outs):
        assert torch.equal(o1, o2) and torch.equal(v1, v2) and torch.equal(s1, s2)


def test_argument_errors_reach_the_caller(zb):
    w = SMALL.replace(dtype="f16", head_dim=128)
    c = GpuCache(zb, w, np.full((2, 2), 4), np.full((2, 2), 4), np.full((2, 2), 1))
    try:
        q, k, v = (t.cuda() for t in wl.decode_inputs(w, 0))
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_decode_step(c.h, 7, q, k, v, c.out_all)
        assert e.value.status == zb.ZSM_ERR_INVALID_ARG
        big = torch.zeros(q.numel() + 8, dtype=q.dtype, device="cuda")
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_decode_step(c.h, -1, big[1:], k, v, c.out_all)          # misaligned pointer
        assert e.value.status == zb.ZSM_ERR_INVALID_ARG
        small = torch.empty(16, dtype=torch.uint8, device="cuda")
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_cache_create(c.cfg, small)
        assert e.value.status in (zb.ZSM_ERR_BUFFER_TOO_SMALL, zb.ZSM_ERR_INVALID_ARG)
        bad = zb.make_config(1, 1, 3, 1, 128, "f16", [4], [4], [1])      # group size 3
        buf = torch.empty(zb.zsm_cache_bytes(bad), dtype=torch.uint8, device="cuda")
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_cache_create(bad, buf)
        assert e.value.status == zb.ZSM_ERR_UNSUPPORTED
    finally:
        c.close()


def test_wrong_tensors_are_refused_before_they_reach_the_device(zb):
    """The binding checks every tensor against the cache's shape: a short, wrongly typed, host
    or non-contiguous tensor raises instead of becoming an out-of-bounds access in a kernel."""
    w = SMALL.replace(dtype="f16", head_dim=128)
    c = GpuCache(zb, w, np.full((2, 2), 4), np.full((2, 2), 4), np.full((2, 2), 1))
    try:
        q, k, v = (t.cuda() for t in wl.decode_inputs(w, 0))
        out = c.out_all
        with pytest.raises(ValueError):
            zb.zsm_decode_step(c.h, -1, q[0], k, v, out)                   # one layer's q for all layers
        with pytest.raises(ValueError):
            zb.zsm_decode_step(c.h, -1, q, k[:, :1], v, out)               # short k_new
        with pytest.raises(TypeError):
            zb.zsm_decode_step(c.h, -1, q.float(), k, v, out)              # wrong dtype
        with pytest.raises(TypeError):
            zb.zsm_decode_step(c.h, -1, q.cpu(), k, v, out)                # host tensor
        with pytest.raises(ValueError):
            zb.zsm_decode_step(c.h, -1, q.transpose(1, 2), k, v, out)      # not contiguous
        with pytest.raises(TypeError):
            zb.zsm_decode_step(c.h, -1, q, k, v, out, victim_pos=torch.zeros(8, device="cuda"))
        with pytest.raises(ValueError):
            zb.zsm_decode_step(c.h, 0, q[0], k[0], v[0], out[0],
                               merge_slot=torch.zeros(1, dtype=torch.int32, device="cuda"))
        T, W = 64, 8
        K = torch.zeros(w.batch, w.n_kv_heads, T, 128, dtype=torch.float16, device="cuda")
        Qw = torch.zeros(w.batch, w.n_q_heads, W, 128, dtype=torch.float16, device="cuda")
        ws = torch.empty(zb.zsm_prefill_workspace_bytes(c.h, T, W), dtype=torch.uint8, device="cuda")
        with pytest.raises(ValueError):
            zb.zsm_prefill_compress(c.h, 0, K[:, :, :32].contiguous(), K, Qw, None, T, W, ws)
        with pytest.raises(ValueError):
            zb.zsm_prefill_compress(c.h, 0, K, K, Qw[:, :1].contiguous(), None, T, W, ws)
        with pytest.raises(TypeError):
            zb.zsm_prefill_compress(c.h, 0, K, K, None, torch.zeros(w.batch, w.n_kv_heads, T,
                                                                    dtype=torch.float16, device="cuda"),
                                    T, 0, ws)
        with pytest.raises(ValueError):
            zb.zsm_prefill_compress(c.h, 0, K, K, Qw, None, T, W, ws,
                                    dbg_targets=torch.zeros(T, dtype=torch.int32, device="cuda"))
        zb.zsm_prefill_compress(c.h, 0, K, K, Qw, None, T, W, ws)          # and the right ones pass
        zb.zsm_decode_step(c.h, -1, q, k, v, out)
        assert c.status() == 0
        assert c.h.buf is c.buf                                            # the handle keeps the buffer
    finally:
        c.close()


def test_bounded_wait_gives_up_and_reports_timeout(zb):
    """The device-side failure detector, run without a fault: a wait that nothing can satisfy
    ends by its time limit, the kernel returns, the sticky status says ZSM_ERR_TIMEOUT, and the
    cache decodes normally afterwards."""
    w = SMALL.replace(dtype="f16", head_dim=128)
    c = GpuCache(zb, w, np.full((2, 2), 4), np.full((2, 2), 4), np.full((2, 2), 1))
    try:
        assert c.status() == 0
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        zb.zsm_selftest_wait_timeout(c.h, 3000)          # 3 ms
        t1.record()
        assert c.status() == zb.ZSM_ERR_TIMEOUT
        assert 2.5 <= t0.elapsed_time(t1) <= 200.0, "the wait must last about its limit, then end"
        assert c.status() == 0                            # reading clears it
        q, k, v = (t.cuda() for t in wl.decode_inputs(w, 0))
        c.decode(q, k, v)
        assert c.status() == 0
        with pytest.raises(zb.ZsmError):
            zb.zsm_selftest_wait_timeout(c.h, 0)
    finally:
        c.close()


def test_scores_of_either_sign_order_as_floats(zb, oracle):
    """Scores handed in from outside (import, caller-supplied prompt scores) may be negative or
    -0.0: the victim is still the lowest float, not the lowest bit pattern; NaN is refused."""
    w = wl.Workload("signed", 1, 1, 2, 1, 128, "f16", 0, 0, 0, None, 19)
    cache = GpuCache(zb, w, [[2]], [[6]], [[2]], lam=1.0)
    stats = ParityStats()
    try:
        rs = np.random.RandomState(7)
        T = 40
        K = torch.from_numpy(rs.randn(T, 128)).to(torch.float16)
        V = torch.from_numpy(rs.randn(T, 128)).to(torch.float16)
        scores = np.linspace(-30.0, 30.0, T).astype(np.float32)
        rs.shuffle(scores)
        scores[5], scores[9] = -0.0, 0.0
        unit = oracle_unit_for(oracle, cache, 0, 0)
        unit.prefill_compress(f64(K), f64(V), scores=scores)
        dbg = cache.prefill(0, K[None, None].cuda(), V[None, None].cuda(), None,
                            torch.from_numpy(scores)[None, None].cuda())
        state_check(unit, cache.export(0, 0, 0), stats, tag="signed scores, prompt pass")
        for step in range(12):
            q, k, v = wl.decode_inputs(w, step)
            out, vic, slot = cache.decode(q.cuda(), k.cuda(), v.cuda())
            oracle_step_check(unit, f64(q)[0, 0], f64(k)[0, 0, 0], f64(v)[0, 0, 0], f64(out)[0, 0],
                              int(vic.cpu()[0, 0, 0]), int(slot.cpu()[0, 0, 0]), w.dtype, stats,
                              tag=f"signed scores step {step}")
        assert stats.selections >= 10 and stats.victim_near_ties == 0
        assert cache.status() == 0
        st = cache.export(0, 0, 0)
        st["score"] = st["score"].copy()
        st["score"][1] = np.nan
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_cache_import_unit(cache.h, 0, 0, 0, 128, st)
        assert e.value.status == zb.ZSM_ERR_INVALID_ARG
        bad = torch.from_numpy(scores.copy())
        bad[3] = float("nan")
        cache.prefill(0, K[None, None].cuda(), V[None, None].cuda(), None, bad[None, None].cuda())
        assert cache.status() == zb.ZSM_ERR_DEVICE_CHECK
    finally:
        cache.close()


def test_caches_of_one_shape_and_different_budgets_coexist(zb):
    """Two live caches that use the same kernel but need different amounts of shared memory:
    creating the second must not lower the launch limit the first one needs."""
    w = wl.Workload("coexist", 1, 1, 2, 2, 128, "f16", 0, 0, 0, None, 18)
    small = GpuCache(zb, w, np.full((1, 2), 8), np.full((1, 2), 8), np.full((1, 2), 1), tune_ctas_per_sm=2)
    big = GpuCache(zb, w, np.full((1, 2), 100), np.full((1, 2), 15000), np.full((1, 2), 4),
                   tune_ctas_per_sm=2)
    try:
        # the large weight array leaves room for fewer ring stages: the two caches ask for
        # different amounts of shared memory
        assert zb.zsm_decode_launch_info(big.h, -1)[2] != zb.zsm_decode_launch_info(small.h, -1)[2]
        q, k, v = (t.cuda() for t in wl.decode_inputs(w, 0))
        for c in (small, big, small, big):
            c.decode(q, k, v)
        assert big.status() == 0 and small.status() == 0
    finally:
        big.close(), small.close()


@pytest.mark.parametrize("ctas,warps", [(1, 16), (1, 5), (2, 8), (2, 3), (3, 4)])
def test_launch_forms_agree(zb, oracle, ctas, warps):
    """The wide form (one CTA per SM, up to sixteen consumer warps whose groups take tiles in
    turn) and the paired form, with warp counts that do and do not tile a stage evenly."""
    w = wl.Workload("forms", 1, 2, 8, 2, 128, "f16", 0, 0, 0, None, 20)
    stats = run_decode(zb, oracle, w, np.array([[30, 60]]), np.array([[150, 41]]), np.array([[3, 5]]),
                       steps=260, check_state_every=130, tune_ctas_per_sm=ctas,
                       tune_consumer_warps=warps)
    assert stats.selections > 300


@pytest.mark.parametrize("cluster,warps", [(2, 16), (4, 16), (8, 16), (4, 5), (8, 3)])
def test_split_forms_agree(zb, oracle, cluster, warps):
    """The split form at every cluster size, with warp counts that do and do not tile a stage
    evenly: slices that end inside a tile, a rank whose share is only the merged slots, the
    victim on any rank."""
    w = wl.Workload("split", 1, 2, 8, 2, 128, "f16", 0, 0, 0, None, 23)
    cache = GpuCache(zb, w, np.array([[30, 60]]), np.array([[150, 41]]), np.array([[3, 40]]),
                     tune_split=cluster, tune_consumer_warps=warps)
    try:
        grid, block, _ = zb.zsm_decode_launch_info(cache.h, -1)
        assert grid == w.batch * w.n_kv_heads * cluster and block == (warps + 2) * 32
    finally:
        cache.close()
    stats = run_decode(zb, oracle, w, np.array([[30, 60]]), np.array([[150, 41]]), np.array([[3, 40]]),
                       steps=260, check_state_every=130, tune_split=cluster,
                       tune_consumer_warps=warps)
    assert stats.selections > 300 and stats.merges > 100


def test_split_form_with_a_large_residual_pool(zb, oracle):
    """More merged slots than rank 0 keeps in shared memory for the residual argmax (they are
    then read from global memory), spanning several fp32 tiles."""
    w = wl.Workload("split_res", 1, 1, 4, 2, 128, "bf16", 0, 0, 0, None, 24)
    stats = run_decode(zb, oracle, w, np.array([[10, 12]]), np.array([[60, 90]]), np.array([[70, 100]]),
                       steps=330, check_state_every=110)
    assert stats.merges > 150


@pytest.mark.parametrize("split", [0, 1])
def test_cosine_slot_similarity(zb, oracle, split):
    """The cosine form of Eq. (hatr) in both decode kernels (heavy-hitter keys are longer than
    ordinary ones, so the two forms do not always agree)."""
    w = wl.Workload("cosine", 1, 2, 4, 2, 128, "f16", 0, 0, 0, None, 27)
    stats = run_decode(zb, oracle, w, np.array([[6, 10]]), np.array([[20, 31]]), np.array([[4, 9]]),
                       steps=220, check_state_every=110, tune_split=split, similarity=1)
    assert stats.merges > 300


@pytest.mark.parametrize("split", [0, 1])
def test_inconsistent_state_is_reported_not_trapped(zb, split):
    """A full pool whose every token claims to sit inside the proximity window has no eviction
    candidate.  The kernel records ZSM_ERR_DEVICE_CHECK in the sticky status word, leaves that
    unit's rows alone (only its token count advances) and keeps running; the healthy unit of
    the same launch decodes as usual; reading the status clears it."""
    w = wl.Workload("badstate", 1, 1, 2, 2, 128, "f16", 0, 0, 0, None, 29)
    cache = GpuCache(zb, w, [[4, 4]], [[4, 4]], [[2, 2]], tune_split=split)
    try:
        rs = np.random.RandomState(4)
        T = 100
        bad = dict(K=rs.randn(8, 128).astype(np.float32), V=rs.randn(8, 128).astype(np.float32),
                   score=np.full(8, 0.1, np.float32), pos=np.full(8, T - 1, np.int32),
                   Kr=rs.randn(2, 128).astype(np.float32), Vr=rs.randn(2, 128).astype(np.float32),
                   w=np.array([3, 5], np.uint32), n_live=8, n_res=2, T=T)
        zb.zsm_cache_import_unit(cache.h, 0, 0, 0, 128, bad)
        q, k, v = (t.cuda() for t in wl.decode_inputs(w, 0))
        out, vic, slot = cache.decode(q, k, v)
        assert cache.status() == zb.ZSM_ERR_DEVICE_CHECK
        assert cache.status() == 0  # sticky until read, then clear
        assert int(vic.cpu()[0, 0, 0]) == -1 and int(slot.cpu()[0, 0, 0]) == -1
        after = cache.export(0, 0, 0)
        np.testing.assert_array_equal(after["pos"], bad["pos"])
        assert after["n_live"] == 8 and after["n_res"] == 2 and after["T"] == T + 1
        np.testing.assert_array_equal(after["w"], bad["w"])
        # the other unit of the launch started empty and took the token
        ok_unit = cache.export(0, 0, 1)
        assert ok_unit["n_live"] == 1 and ok_unit["T"] == 1
        assert torch.isfinite(out.float()).all()
        # and the cache goes on working
        cache.decode(q, k, v)
        assert cache.status() == zb.ZSM_ERR_DEVICE_CHECK  # the bad unit is still bad ...
        ok_unit = cache.export(0, 0, 1)
        assert ok_unit["n_live"] == 2 and ok_unit["T"] == 2  # ... the good one is not held up
    finally:
        cache.close()
