"""zsm_prefill_compress_static: the prompt pass for callers that cannot allocate device memory
when they call (a server whose memory pool already holds the whole GPU, a loop that cannot
afford an allocation's synchronisation).  Its scratch is a fixed array inside the library, so
the only thing that can differ from zsm_prefill_compress is where the scratch lives: every
result must be identical to the workspace entry point's, also on a second call that finds the
first call's leftovers in the array.  Collected last on purpose (file name)."""
import numpy as np
import pytest
import torch

import workloads as wl
from harness import GpuCache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import binding
    return binding


def _state(cache, w):
    out = []
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            for layer in range(w.n_layers):
                out.append(cache.export(layer, b, h))
    return out


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(zb):
    w = wl.Workload("noalloc", 2, 2, 4, 2, 128, "f16", 700, 0, 24, None, 31)
    bp = np.array([[16, 40], [8, 33]])
    bc = np.array([[20, 61], [9, 70]])
    br = np.array([[2, 5], [1, 9]])
    ref, sta = GpuCache(zb, w, bp, bc, br), GpuCache(zb, w, bp, bc, br)
    try:
        assert zb.zsm_prefill_workspace_bytes(sta.h, w.prompt_len, w.window) <= zb.ZSM_STATIC_SCRATCH_BYTES
        # two calls in a row, on different inputs: the second finds the first one's leftovers
        for layer in range(w.n_layers):
            K, V, Qw = (t.cuda() for t in wl.prompt(w, layer))
            d_ref = ref.prefill(layer, K, V, Qw)
            T, W = K.shape[2], Qw.shape[2]
            d_sta = {"scores": torch.empty_like(d_ref["scores"]),
                     "evicted": torch.zeros_like(d_ref["evicted"]),
                     "targets": torch.full_like(d_ref["targets"], -9)}
            zb.zsm_prefill_compress_static(sta.h, layer, K, V, Qw, None, T, W, d_sta["scores"],
                                           d_sta["evicted"], d_sta["targets"])
            torch.cuda.synchronize()
            for key in d_ref:
                assert torch.equal(d_ref[key], d_sta[key]), f"layer {layer}: {key} differs"
        assert ref.status() == 0 and sta.status() == 0
        for a, b in zip(_state(ref, w), _state(sta, w)):
            assert (a["n_live"], a["n_res"], a["T"]) == (b["n_live"], b["n_res"], b["T"])
            for key in ("K", "V", "score", "pos", "Kr", "Vr", "w"):
                np.testing.assert_array_equal(a[key], b[key], err_msg=key)
        # the caller-supplied-scores form shares the array too
        scores = torch.rand(w.batch, w.n_kv_heads, w.prompt_len, device="cuda") + 1e-3
        K, V, _ = (t.cuda() for t in wl.prompt(w, 0))
        ref.prefill(0, K, V, None, scores)
        zb.zsm_prefill_compress_static(sta.h, 0, K, V, None, scores, w.prompt_len, 0)
        for a, b in zip(_state(ref, w), _state(sta, w)):
            for key in ("K", "V", "score", "pos", "Kr", "Vr", "w"):
                np.testing.assert_array_equal(a[key], b[key], err_msg=key)
    finally:
        ref.close(), sta.close()


def test_static_scratch_call_leaves_device_memory_alone(zb):
    """What the entry point is for: once a cache exists on the device (its creation does the
    one-time look-up of the array, which is when the device reserves the array's bytes), a call
    changes neither the free device memory nor what torch's allocator holds."""
    w = wl.Workload("noalloc_mem", 1, 2, 4, 2, 128, "f16", 500, 0, 16, None, 33)
    c = GpuCache(zb, w, np.full((1, 2), 16), np.full((1, 2), 20), np.full((1, 2), 3))
    try:
        K, V, Qw = (t.cuda() for t in wl.prompt(w, 0))
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        reserved0 = torch.cuda.memory_reserved()
        for _ in range(3):
            zb.zsm_prefill_compress_static(c.h, 0, K, V, Qw, None, w.prompt_len, w.window)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0, f"free device memory changed by {free0 - free1} bytes"
        assert torch.cuda.memory_reserved() == reserved0
        assert c.status() == 0
    finally:
        c.close()


def test_prompt_beyond_the_fixed_scratch_is_refused(zb):
    w = wl.Workload("noalloc_big", 1, 4, 8, 8, 128, "f16", 0, 0, 0, None, 32)
    c = GpuCache(zb, w, np.full((1, 8), 8), np.full((1, 8), 8), np.full((1, 8), 1))
    try:
        T, W = 40000, 32       # 32 units x 40000 x (13 + 128) bytes > 16 MiB
        assert zb.zsm_prefill_workspace_bytes(c.h, T, W) > zb.ZSM_STATIC_SCRATCH_BYTES
        tiny = torch.zeros(16, dtype=torch.float16, device="cuda")   # never read: refused on the host
        with pytest.raises(zb.ZsmError) as e:
            zb.zsm_prefill_compress_static(c.h, 0, tiny, tiny, tiny, None, T, W)
        assert e.value.status == zb.ZSM_ERR_BUFFER_TOO_SMALL
        assert c.status() == 0
    finally:
        c.close()
