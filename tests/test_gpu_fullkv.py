"""Uncompressed decode attention (the FullKV comparator) against its definition: softmax(q K^T /
sqrt(d)) V, evaluated by torch SDPA in fp64 on the CPU.  Shapes span several chunks with ragged
last chunks and tiles, both head dimensions, grouped queries, both 16-bit types."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import binding
    return binding


def reference(K, V, q, scale=None):
    G = q.shape[1]
    Kd, Vd = K.double().cpu(), V.double().cpu()
    o = torch.nn.functional.scaled_dot_product_attention(q.double().cpu(), Kd, Vd, scale=scale)
    return o                                                  # [units, G, d]: G queries share K, V


def run(zb, units, T, d, G, dtype, seed, scale=0.0, boost=3.0):
    g = torch.Generator().manual_seed(seed)
    u = torch.randn(d, generator=g)
    u /= u.norm()
    K = torch.randn(units, T, d, generator=g)
    K[:, ::37] += boost * u                                   # a few heavy hitters
    V = torch.randn(units, T, d, generator=g)
    q = torch.randn(units, G, d, generator=g) + boost * u
    K, V, q = (t.to(dtype).cuda() for t in (K, V, q))
    out = torch.empty_like(q)
    ws = torch.empty(zb.zsm_fullkv_workspace_bytes(units, G, d, T), dtype=torch.uint8, device="cuda")
    zb.zsm_fullkv_decode(K, V, q, out, ws, softmax_scale=scale)
    assert zb.zsm_fullkv_status(ws) == 0
    ref = reference(K, V, q, scale if scale > 0 else None)
    torch.testing.assert_close(out.double().cpu(), ref, atol=2e-3, rtol=1e-2)
    return out


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("d,G", [(128, 1), (128, 4), (64, 2), (64, 8), (128, 8)])
def test_matches_softmax_attention(zb, dtype, d, G):
    run(zb, units=5, T=9000 // G + 77, d=d, G=G, dtype=dtype, seed=3 + d + G)


@pytest.mark.parametrize("T", [1, 15, 16, 17, 63, 64, 65, 4095, 4096, 4097, 8200])
def test_lengths_around_tile_and_chunk_edges(zb, T):
    run(zb, units=3, T=T, d=128, G=1, dtype=torch.float16, seed=T)


def test_many_units_and_custom_scale(zb):
    run(zb, units=700, T=300, d=128, G=2, dtype=torch.bfloat16, seed=9, scale=0.05)


def test_agrees_with_the_compressed_path_when_nothing_is_evicted(zb):
    """Same inputs through zsm_decode_step on a cache whose budget holds the whole history and
    through the uncompressed kernel: both are plain softmax attention."""
    import workloads as wl
    from harness import GpuCache
    w = wl.Workload("fk", 1, 2, 8, 2, 128, "f16", 0, 0, 0, None, 19)
    steps = 90
    c = GpuCache(zb, w, np.full((1, 2), 10), np.full((1, 2), steps), np.full((1, 2), 2))
    try:
        ks, vs = [], []
        for s in range(steps):
            q, k, v = (t.cuda() for t in wl.decode_inputs(w, s))
            out, _, _ = c.decode(q, k, v)
            ks.append(k[0]), vs.append(v[0])
        K = torch.stack(ks, dim=2).reshape(4, steps, 128).contiguous()      # [b*h, T, d]
        V = torch.stack(vs, dim=2).reshape(4, steps, 128).contiguous()
        qq = q[0].reshape(4, 4, 128).contiguous()
        o2 = torch.empty_like(qq)
        ws = torch.empty(zb.zsm_fullkv_workspace_bytes(4, 4, 128, steps), dtype=torch.uint8, device="cuda")
        zb.zsm_fullkv_decode(K, V, qq, o2, ws)
        assert zb.zsm_fullkv_status(ws) == 0
        torch.testing.assert_close(o2.float(), out[0].reshape(4, 4, 128).float(), atol=2e-3, rtol=1e-2)
    finally:
        c.close()


def test_bad_arguments(zb):
    K = torch.zeros(2, 10, 128, dtype=torch.float32, device="cuda")
    q = torch.zeros(2, 1, 128, dtype=torch.float32, device="cuda")
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(zb.ZsmError) as e:
        zb.zsm_fullkv_decode(K, K, q, q.clone(), ws)
    assert e.value.status == zb.ZSM_ERR_UNSUPPORTED          # fp32 storage
    Kh, qh = K.half(), q.half()
    with pytest.raises(zb.ZsmError) as e:
        zb.zsm_fullkv_decode(Kh, Kh, qh, qh.clone(), ws[:64])
    assert e.value.status == zb.ZSM_ERR_BUFFER_TOO_SMALL
    with pytest.raises(zb.ZsmError):
        zb.zsm_fullkv_workspace_bytes(2, 3, 128, 10)          # group size 3
