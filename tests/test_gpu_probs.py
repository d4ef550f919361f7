"""Probability pipeline kernel (guidance, temperature, top-k with ties, softmax) against the oracle's."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_18183_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx16k():
    # any bf16 context with a 16384-entry vocabulary: the pipeline only needs V
    sh = synth.ModelShape(1, 64, 1, 64, 16384, 4, 4, 3, "bf16")
    c = binding.Context(sh, synth.make_weights(sh, 3, target_entropy=None), 2, 4)
    yield c
    c.hbsjd_destroy()


def _check(ctx, lc, lu, s, tau, k):
    import torch
    p = ctx.hbsjd_probs(torch.from_numpy(lc).cuda(), None if lu is None else torch.from_numpy(lu).cuda(), s, tau,
                        k).cpu().numpy()
    for r in range(lc.shape[0]):
        ref = O.probs(lc[r], None if lu is None else lu[r], s=s, tau=tau, k=k)
        # the same support exactly (the threshold is found exactly, ties kept); entries whose probability
        # underflows fp32 may be flushed to zero by expf
        big = ref > 1e-30
        np.testing.assert_array_equal(p[r][big] > 0, ref[big] > 0)
        assert p[r][ref == 0].max(initial=0.0) < 1e-37  # dropped entries are exactly 0; underflow aside
        # ... and the same values up to expf / fp32-sum rounding
        assert np.abs(p[r] - ref).max() <= 1e-6 + 1e-5 * ref.max()
        assert np.all(np.abs(p[r] - ref) <= 1e-6 + 1e-5 * ref)
        assert abs(float(p[r].astype(np.float64).sum()) - 1.0) < 1e-4


@pytest.mark.parametrize("k", [0, 1, 7, 1000, 16383, 16384, 20000])
def test_gaussian_logits(ctx16k, k):
    rng = np.random.default_rng(k)
    lc = (rng.normal(size=(6, 16384)) * 3.5).astype(np.float32)
    lu = (rng.normal(size=(6, 16384)) * 3.5).astype(np.float32)
    _check(ctx16k, lc, None, 1.0, 1.0, k)
    _check(ctx16k, lc, lu, 4.0, 0.7, k)


def test_ties_and_crowded_bins(ctx16k):
    """Heavily tied logits: the k-th value is shared by thousands of entries (all kept), one bin of the
    selection histogram holds nearly everything (the radix fallback runs), and constant rows keep all."""
    rng = np.random.default_rng(1)
    V = 16384
    rows = []
    rows.append(np.round(rng.normal(size=V) * 2).astype(np.float32))           # ~10 distinct values
    rows.append(np.where(rng.random(V) < 0.001, 50.0, rng.normal(size=V) * 1e-3).astype(np.float32))  # outliers
    rows.append(np.full(V, 1.25, dtype=np.float32))                              # constant
    r3 = rng.normal(size=V).astype(np.float32)
    r3[:3000] = r3[5]                                                            # a 3000-way tie
    rows.append(r3)
    r4 = (rng.normal(size=V) * 1e-6 + 7.0).astype(np.float32)                    # adjacent floats
    rows.append(r4)
    rows.append(-np.abs(rng.normal(size=V)).astype(np.float32) * 30)             # negative, wide
    lc = np.stack(rows)
    for k in (1, 5, 1000, 4000, 16000):
        _check(ctx16k, lc, None, 1.0, 1.0, k)
