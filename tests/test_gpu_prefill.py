"""GPU parity of the one-shot prompt compression and of prompt pass + decode end to end
(workloads c1 and c2 in full) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import workloads as wl
from harness import (GpuCache, ParityStats, f64, oracle_step_check, prefill_check, split_budgets,
                     state_check)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import binding
    return binding


def prefill_all_units(zb, oracle, w, cache, layer, stats, scores=None):
    K, V, Qw = wl.prompt(w, layer)
    if scores is None:
        dbg = cache.prefill(layer, K.cuda(), V.cuda(), Qw.cuda())
    else:
        dbg = cache.prefill(layer, K.cuda(), V.cuda(), None, scores.cuda())
    units = {}
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            units[(layer, b, h)] = prefill_check(
                oracle, cache, layer, b, h, K, V, Qw, dbg, stats,
                scores_given=None if scores is None else scores[b, h].numpy(),
                tag=f"prompt pass unit {(layer, b, h)}")
    return units


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("head_dim,group", [(64, 1), (128, 1), (128, 4), (64, 2)])
def test_prompt_pass_all_kernel_variants(zb, oracle, dtype, head_dim, group):
    """Scores, selection, merge chain and gathered state for every kernel variant; prompt of
    several score chunks with a ragged tail; ragged per-head budgets."""
    w = wl.Workload("pp", 2, 2, 2 * group, 2, head_dim, dtype, 700, 0, 24, None, 21)
    bp = np.array([[16, 40], [8, 33]])
    bc = np.array([[20, 61], [9, 70]])
    br = np.array([[2, 5], [1, 9]])
    cache = GpuCache(zb, w, bp, bc, br)
    stats = ParityStats()
    try:
        for layer in range(w.n_layers):
            prefill_all_units(zb, oracle, w, cache, layer, stats)
        assert cache.status() == 0
    finally:
        cache.close()
    assert stats.selections > 4000 and stats.merges > 3500


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("head_dim,group,window", [(128, 1, 32), (64, 2, 32), (128, 4, 24), (128, 4, 32),
                                                   (64, 1, 64)])
def test_prompt_pass_window_scoring_on_tcgen05(zb, oracle, dtype, head_dim, group, window):
    """Windows of G * W = 32, 64, 96 and 128 query rows take the tcgen05 form of the window
    scoring (one, two, three and four blocks of 32 rows per chunk; both accumulators, both chunk
    stages and every barrier phase wrap: 11 chunks over at most 3 CTAs per unit here); the prompt
    ends inside a chunk.  Scores, selection, merge targets and state against the oracle."""
    w = wl.Workload("pptc", 1, 2, 2 * group, 2, head_dim, dtype, 1333, 0, window, None, 45)
    bp = np.array([[16, 40]])
    bc = np.array([[20, 61]])
    br = np.array([[2, 5]])
    cache = GpuCache(zb, w, bp, bc, br)
    stats = ParityStats()
    try:
        prefill_all_units(zb, oracle, w, cache, 0, stats)
        assert cache.status() == 0
    finally:
        cache.close()
    assert stats.selections > 4000


@pytest.mark.parametrize("T,window", [(5, 5), (30, 8), (48, 48), (129, 1), (300, 300)])
def test_prompt_lengths_around_the_budgets(zb, oracle, T, window):
    """Prompts shorter than B_p, shorter than B_p + B_c (nothing evicted), barely longer
    (residual slots only partly filled), and a full-history window (W = T)."""
    w = wl.Workload("len", 1, 1, 2, 2, 128, "f16", T, 0, window, None, 22)
    cache = GpuCache(zb, w, [[10, 20]], [[25, 100]], [[4, 40]])
    stats = ParityStats()
    try:
        prefill_all_units(zb, oracle, w, cache, 0, stats)
        assert cache.status() == 0
    finally:
        cache.close()


@pytest.mark.parametrize("budgets", [(0, 12, 2), (10, 0, 4), (6, 9, 0), (1, 1, 1)])
def test_prompt_pass_degenerate_budgets(zb, oracle, budgets):
    w = wl.Workload("deg", 1, 2, 2, 1, 64, "bf16", 200, 0, 16, None, 23)
    cache = GpuCache(zb, w, [[budgets[0]]], [[budgets[1]]], [[budgets[2]]])
    stats = ParityStats()
    try:
        prefill_all_units(zb, oracle, w, cache, 0, stats)
    finally:
        cache.close()


@pytest.mark.parametrize("br", [3, 33, 100, 150])
def test_residual_pool_sizes(zb, oracle, br):
    """Residual pools on both sides of the sizes at which the merge kernel changes form: the
    blocked form with one or two slots per lane of its chain warp (B_r <= 32, 64), merged keys
    in registers with four rows per thread (B_r <= 128), in shared memory beyond that."""
    w = wl.Workload("pool", 1, 1, 2, 2, 128, "f16", 1500, 0, 16, None, 25)
    cache = GpuCache(zb, w, [[40, 64]], [[60, 90]], [[br, max(1, br // 2)]])
    stats = ParityStats()
    try:
        prefill_all_units(zb, oracle, w, cache, 0, stats)
        assert cache.status() == 0 and stats.merges > 2000
    finally:
        cache.close()


def test_layer_with_more_units_than_resident_ctas(zb, oracle):
    """320 units in one layer: more chains than the GPU holds CTAs of the row-per-warp merge
    kernel, so the one-warp form runs; every unit is checked."""
    w = wl.Workload("many", 1, 40, 8, 8, 64, "bf16", 260, 0, 8, None, 26)
    cache = GpuCache(zb, w, np.full((1, 8), 12), np.full((1, 8), 20), np.arange(1, 9).reshape(1, 8) * 4)
    stats = ParityStats()
    try:
        prefill_all_units(zb, oracle, w, cache, 0, stats)
        assert cache.status() == 0 and stats.merges > 40000
    finally:
        cache.close()


def test_prompt_passes_on_four_streams_repeat_the_serial_result(zb):
    """Eight layers' prompt passes round-robin on four streams, three times over, against the
    same layers compressed one after another: scores, eviction flags and merge targets must be
    bit-identical (every kernel of the pass is deterministic).  The window scoring kernel's
    write-out warps run at uneven pace when launches of several streams share the SMs."""
    w = wl.Workload("four", 8, 1, 8, 8, 128, "f16", 6000, 0, 32, None, 46)
    bp, bc, br = np.full((8, 8), 40), np.full((8, 8), 60), np.full((8, 8), 4)
    cache = GpuCache(zb, w, bp, bc, br)
    try:
        T = w.prompt_len
        dev = [[t.cuda() for t in wl.prompt(w, layer)] for layer in range(w.n_layers)]

        def outputs():
            return {"scores": torch.empty(w.batch, w.n_kv_heads, T, dtype=torch.float32, device="cuda"),
                    "evicted": torch.zeros(w.batch, w.n_kv_heads, T, dtype=torch.uint8, device="cuda"),
                    "targets": torch.full((w.batch, w.n_kv_heads, T), -9, dtype=torch.int32, device="cuda")}

        need = zb.zsm_prefill_workspace_bytes(cache.h, T, w.window)
        wss = [torch.empty(need, dtype=torch.uint8, device="cuda") for _ in range(4)]
        serial = []
        for layer in range(w.n_layers):
            d = outputs()
            K, V, Qw = dev[layer]
            zb.zsm_prefill_compress(cache.h, layer, K, V, Qw, None, T, w.window, wss[0], d["scores"],
                                    d["evicted"], d["targets"])
            serial.append(d)
        torch.cuda.synchronize()
        streams = [torch.cuda.Stream() for _ in range(4)]
        for rep in range(3):
            side = []
            for layer in range(w.n_layers):
                d = outputs()
                K, V, Qw = dev[layer]
                zb.zsm_prefill_compress(cache.h, layer, K, V, Qw, None, T, w.window, wss[layer % 4],
                                        d["scores"], d["evicted"], d["targets"], stream=streams[layer % 4])
                side.append(d)
            torch.cuda.synchronize()
            assert cache.status() == 0
            for layer in range(w.n_layers):
                for key in ("scores", "evicted", "targets"):
                    assert torch.equal(side[layer][key], serial[layer][key]), (rep, layer, key)
    finally:
        cache.close()


def test_layers_compressed_side_by_side_on_two_streams(zb, oracle):
    """Layers are independent: their prompt passes may run at the same time on different
    streams, each with a workspace of its own.  Three layers on two streams (the third queues
    behind the first), every unit of every layer checked against the oracle."""
    w = wl.Workload("side", 3, 2, 4, 2, 128, "f16", 1800, 0, 16, None, 40)
    bp, bc, br = np.full((3, 2), 24), np.full((3, 2), 40), np.array([[3, 40], [9, 5], [70, 2]])
    cache = GpuCache(zb, w, bp, bc, br)
    stats = ParityStats()
    try:
        streams = [torch.cuda.Stream() for _ in range(2)]
        need = zb.zsm_prefill_workspace_bytes(cache.h, w.prompt_len, w.window)
        wss = [torch.empty(need, dtype=torch.uint8, device="cuda") for _ in range(2)]
        prompts = [wl.prompt(w, layer) for layer in range(w.n_layers)]
        dev = [[t.cuda() for t in pr] for pr in prompts]
        dbgs = []
        torch.cuda.synchronize()
        for layer in range(w.n_layers):
            T = w.prompt_len
            d = {"scores": torch.empty(w.batch, w.n_kv_heads, T, dtype=torch.float32, device="cuda"),
                 "evicted": torch.zeros(w.batch, w.n_kv_heads, T, dtype=torch.uint8, device="cuda"),
                 "targets": torch.full((w.batch, w.n_kv_heads, T), -9, dtype=torch.int32, device="cuda")}
            K, V, Qw = dev[layer]
            zb.zsm_prefill_compress(cache.h, layer, K, V, Qw, None, T, w.window, wss[layer % 2],
                                    d["scores"], d["evicted"], d["targets"], stream=streams[layer % 2])
            dbgs.append(d)
        torch.cuda.synchronize()
        for layer in range(w.n_layers):
            K, V, Qw = prompts[layer]
            for b in range(w.batch):
                for h in range(w.n_kv_heads):
                    prefill_check(oracle, cache, layer, b, h, K, V, Qw, dbgs[layer], stats,
                                  tag=f"side by side, unit {(layer, b, h)}")
        assert cache.status() == 0 and stats.merges > 15000
    finally:
        cache.close()


def test_supplied_scores_with_exact_ties(zb, oracle):
    """Scores given by the caller, drawn from four values only: the selection is decided by
    the position rule almost everywhere and must match the oracle bit for bit (no near tie
    can exist between distinct values this far apart)."""
    w = wl.Workload("ties", 1, 2, 2, 2, 128, "f16", 1000, 0, 0, None, 24)
    g = torch.Generator().manual_seed(1)
    scores = torch.randint(1, 5, (2, 2, 1000), generator=g).float() * 0.25
    cache = GpuCache(zb, w, [[50, 64]], [[70, 300]], [[3, 12]])
    stats = ParityStats()
    try:
        prefill_all_units(zb, oracle, w, cache, 0, stats, scores=scores)
        assert stats.victim_near_ties == 0
    finally:
        cache.close()


def pipeline(zb, oracle, w, layer_mode=-1, check_state_every=64):
    """Prompt pass for every layer, then every decode step, every unit checked at every step."""
    bp, bc, br = split_budgets(zb, wl.head_budgets(w))
    cache = GpuCache(zb, w, bp, bc, br)
    stats = ParityStats()
    try:
        units = {}
        for layer in range(w.n_layers):
            units.update(prefill_all_units(zb, oracle, w, cache, layer, stats))
        G = w.group
        for step in range(w.decode_steps):
            q, k, v = wl.decode_inputs(w, step)
            out, vic, slot = cache.decode(q.cuda(), k.cuda(), v.cuda(), layer=layer_mode)
            out_h, vic_h, slot_h = f64(out), vic.cpu().numpy(), slot.cpu().numpy()
            q64, k64, v64 = f64(q), f64(k), f64(v)
            for (l, b, h), unit in units.items():
                oracle_step_check(unit, q64[l, b, h * G:(h + 1) * G], k64[l, b, h], v64[l, b, h],
                                  out_h[l, b, h * G:(h + 1) * G], vic_h[l, b, h], slot_h[l, b, h],
                                  w.dtype, stats, tag=f"{w.name} step {step} unit {(l, b, h)}")
            if (step + 1) % check_state_every == 0 or step == w.decode_steps - 1:
                for (l, b, h), unit in units.items():
                    state_check(unit, cache.export(l, b, h), stats, tag=f"{w.name} step {step}")
        assert cache.status() == 0
    finally:
        cache.close()
    assert stats.exact_tie_breaches == 0
    return stats


def test_workload_c1_full(zb, oracle):
    """c1: 1 layer, 4 heads, d 64, fp32, prompt 512 scored with its full history, budget 64,
    64 decode steps: every unit, every step."""
    stats = pipeline(zb, oracle, wl.C1)
    assert stats.steps == 4 * 64 and stats.merges >= 4 * 64
    print("c1", stats)


def test_workload_c2_full(zb, oracle):
    """c2: LLaMA2-7B layer shape, fp16, prompt 4096, budget 205, 256 decode steps: every
    unit, every step; expected near-tie events: none or a handful."""
    stats = pipeline(zb, oracle, wl.C2)
    assert stats.steps == 32 * 256
    assert stats.victim_near_ties + stats.merge_near_ties <= 64
    print("c2", stats)


@pytest.mark.parametrize("br", [5, 70])
def test_prompt_pass_cosine_slot_similarity(zb, oracle, br):
    """The cosine form of Eq. (hatr) in the prompt pass (general merge kernel whatever B_r)."""
    w = wl.Workload("ppcos", 1, 1, 4, 2, 128, "bf16", 900, 0, 16, None, 28)
    cache = GpuCache(zb, w, [[20, 32]], [[30, 50]], [[br, br + 3]], similarity=1)
    stats = ParityStats()
    try:
        prefill_all_units(zb, oracle, w, cache, 0, stats)
        assert cache.status() == 0 and stats.merges > 1000
    finally:
        cache.close()


def test_residual_pool_of_two_rows_per_thread_fp32(zb, oracle):
    """fp32 storage has no blocked form: 33..64 merged slots run the register form with two rows
    per thread."""
    w = wl.Workload("pool32", 1, 1, 2, 2, 64, "f32", 900, 0, 16, None, 30)
    cache = GpuCache(zb, w, [[30, 40]], [[40, 50]], [[40, 64]])
    stats = ParityStats()
    try:
        prefill_all_units(zb, oracle, w, cache, 0, stats)
        assert cache.status() == 0 and stats.merges > 1200
    finally:
        cache.close()
