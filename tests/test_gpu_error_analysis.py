"""The paper's numerical error analysis (Sec. 4.3) on synthetic heavy-hitter data: at 50, 20,
10 and 5 % cache the attention output with residual merging is closer to full attention than
with pure eviction.  The paper gives neither data nor protocol, so the ordering is what is
checked, not its printed values."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_merging_beats_eviction_at_every_ratio():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import error_analysis
    res = error_analysis.run(prompt_len=2048, steps=64)
    print(res)
    for ratio, r in res.items():
        assert 0.0 < r["merge"] < r["evict"], f"ratio {ratio}: merge {r['merge']:.3e} evict {r['evict']:.3e}"
    # less cache, more error, for both policies
    ratios = sorted(res, reverse=True)
    for a, b in zip(ratios, ratios[1:]):
        assert res[a]["evict"] < res[b]["evict"] and res[a]["merge"] < res[b]["merge"]


def test_compensation_term_is_what_makes_merging_pay():
    """Sensitivity axis alpha (App. C.2 / Sec. 3.5): with alpha = 0 a merged slot weighs like one
    token and the output error is close to eviction's; alpha = 1 cuts it several-fold."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import error_analysis
    kw = dict(ratios=(0.1,), prompt_len=2048, steps=48)
    e1 = error_analysis.run(alpha=1.0, **kw)[0.1]
    e0 = error_analysis.run(alpha=0.0, **kw)[0.1]
    assert e1["merge"] < 0.6 * e0["merge"] and e0["merge"] > 0.8 * e0["evict"]


def test_cosine_similarity_variant_runs_through_the_same_kernels():
    """Sensitivity axis "slot similarity" (the cosine form beside Eq. (hatr)): merging still
    beats eviction, and the figure is its own (the variant is not silently the default)."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2503_10714_b200 import error_analysis
    kw = dict(ratios=(0.1,), prompt_len=2048, steps=48)
    dot = error_analysis.run(similarity=0, **kw)[0.1]
    cos = error_analysis.run(similarity=1, **kw)[0.1]
    assert 0.0 < cos["merge"] < cos["evict"]
    assert cos["evict"] == dot["evict"] and cos["merge"] != dot["merge"]
