"""Router scoring head on the GPU (through the C ABI) against the oracle, element by element.

Tolerance: the logit is an fp32 sum of `hidden` exact bf16 x bf16 products (relative error of the
sum about 1e-6 sqrt(hidden) of its terms' magnitude), the sigmoid has slope <= 1/4 and the fast
exponential is good to a few ulp, so 1e-4 absolute on a score in [0, 1] leaves two orders of
magnitude; the selection (an integer) is then taken from the GPU's scores on both sides."""
import numpy as np
import pytest

from oracle.cache import AdapterCache, select_adapter
from oracle.router import router_scores
from paper_2507_01438_b200 import binding as B
from paper_2507_01438_b200 import workloads as wl
from gpu_helpers import to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("Bn,n,hidden,with_bias", [
    (1, 1, 8, False), (1, 1000, 4096, True), (3, 37, 264, True), (8, 2000, 4096, False),
    (11, 129, 1024, True), (20, 513, 2048, False),
])
def test_scores_match_the_oracle(Bn, n, hidden, with_bias):
    import torch
    rng = np.random.Generator(np.random.PCG64(Bn * 1000 + n))
    Wr = wl.normal_bf16(rng, (n, hidden), 2.0 / np.sqrt(hidden))
    h = wl.normal_bf16(rng, (Bn, hidden), 1.0)
    bias = rng.normal(0, 1, size=n).astype(np.float32) if with_bias else None
    got = B.edgelora_router_scores(to_dev_bf16(Wr), torch.from_numpy(bias).cuda() if with_bias else None,
                                   to_dev_bf16(h)).cpu().numpy()
    ref = router_scores(Wr, bias, h)
    assert got.shape == ref.shape and np.all(np.isfinite(got))
    assert np.max(np.abs(got - ref)) <= 1e-4, np.max(np.abs(got - ref))
    if ref.size > 10:
        assert ref.std() > 0.1    # the scores are spread out: a constant output would fail


def test_saturation_and_empty_batch():
    import torch
    Wr = wl.f32_to_bf16_bits(np.array([[100.0] * 16, [-100.0] * 16, [0.0] * 16], dtype=np.float32))
    h = wl.f32_to_bf16_bits(np.ones((2, 16), dtype=np.float32))
    s = B.edgelora_router_scores(to_dev_bf16(Wr), None, to_dev_bf16(h)).cpu().numpy()
    assert np.array_equal(s, np.array([[1.0, 0.0, 0.5]] * 2, dtype=np.float32))
    empty = torch.empty((0, 16), dtype=torch.bfloat16, device="cuda")
    out = B.edgelora_router_scores(to_dev_bf16(Wr), None, empty)
    assert tuple(out.shape) == (0, 3)
    with pytest.raises(B.EdgeLoraError):
        B.edgelora_router_scores(torch.zeros((4, 12), dtype=torch.bfloat16, device="cuda"), None,
                                 torch.zeros((1, 12), dtype=torch.bfloat16, device="cuda"))


def test_scores_drive_the_cache_aware_selection():
    rng = np.random.Generator(np.random.PCG64(77))
    n, hidden = 400, 1024
    Wr = wl.normal_bf16(rng, (n, hidden), 3.0 / np.sqrt(hidden))
    h = wl.normal_bf16(rng, (30, hidden), 1.0)
    scores = B.edgelora_router_scores(to_dev_bf16(Wr), None, to_dev_bf16(h)).cpu().numpy()
    cache, ref = B.edgelora_cache_create(8), AdapterCache(8)
    try:
        hits = 0
        for b in range(30):
            got = B.edgelora_cache_select(cache, np.ascontiguousarray(scores[b]), 3)
            assert got == select_adapter(ref, scores[b], 3)
            hits += got[2]
    finally:
        B.edgelora_cache_destroy(cache)
