"""Checks at full size: workload L (24 layers, dim 1024, vocabulary 16384, batch 128 with guidance = 256 physical
rows, window 32 -> 8192 token rows per forward, the launch configuration bench.py times) and the other full-size
configurations B (12 layers, no guidance), XL (36 layers, 24 x 24 tokens) and stress (L shape, batch 256, bimodal
prefix lengths).

The oracle needs up to half a minute per image-round at these sizes, so element-wise parity is taken on sampled
outputs: one image (the one with the shortest prefix) is followed in lockstep for two rounds while the GPU runs
the whole batch shape; everything else is checked through properties that hold at any size."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_18183_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=["L", "B", "XL", "stress"])
def big(request):
    w = synth.WORKLOADS[request.param]
    weights = G.weights_for(w)
    ctx = binding.Context(w.shape, weights, w.batch, w.window)
    toks, k, lab = synth.make_inputs(w)
    yield w, weights, ctx, toks, k, lab
    ctx.hbsjd_destroy()


def test_fullsize_properties(big):
    w, weights, ctx, toks, k, lab = big
    T = w.shape.T
    outs, stats = [], []
    for mode, gamma in [(binding.EXEC_FULL, 0), (binding.EXEC_COMPACT, 0), (binding.EXEC_HYBRID, w.batch // 2)]:
        out, st = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 17, exec_mode=mode, gamma=gamma))
        outs.append(out.cpu().numpy())
        stats.append(st)
    ref = outs[0]
    # execution modes only choose which rows are physically run: identical tokens, rounds and commits
    for o, st in zip(outs[1:], stats[1:]):
        np.testing.assert_array_equal(o, ref)
        assert st["rounds"] == stats[0]["rounds"] and st["image_forwards"] == stats[0]["image_forwards"]
    assert stats[0]["compact_rounds"] == 0 and stats[1]["full_rounds"] == 0
    assert stats[2]["full_rounds"] > 0 and stats[2]["compact_rounds"] > 0
    assert ref.min() >= 0 and ref.max() < w.shape.vocab
    for b in range(w.batch):
        np.testing.assert_array_equal(ref[b, :k[b]], toks[b, :k[b]])
    assert stats[0]["committed"] == int((T - k).sum())
    # every image commits at least one token per round it is live: rounds <= longest suffix
    assert stats[0]["rounds"] <= int((T - k).max())
    acc = stats[0]["committed"] / stats[0]["image_forwards"]
    assert 1.0 <= acc <= w.window
    # the same seed reproduces the same rollout; another seed does not
    again, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 17, exec_mode=binding.EXEC_HYBRID,
                                                                                 gamma=w.batch // 4))
    np.testing.assert_array_equal(again.cpu().numpy(), ref)
    other, _ = ctx.hbsjd_rollout(G.dev(toks), G.dev(k), G.dev(lab), G.gpu_params(w, 18))
    assert not np.array_equal(other.cpu().numpy(), ref)


def test_fullsize_sampled_image_in_lockstep_with_the_oracle(big):
    w, weights, ctx, toks, k, lab = big
    b = int(np.argmin(k))  # shortest prefix: cheapest prefill for the oracle
    model = O.Model(w.shape, weights)
    rep = G.lockstep(ctx, model, w, toks, k, lab, 23, image_ids=[b], max_rounds=2)
    std, tol = G.bf16_logit_tol(rep["logit_std"], w.shape.n_layers)
    assert rep["max_logit_err"] <= tol, (rep["max_logit_err"], tol)
    assert rep["abs_err_sum"] / rep["abs_err_n"] <= std, (rep["abs_err_sum"] / rep["abs_err_n"], std)
    assert rep["max_p_err"] <= 1e-6
    assert rep["replay_mismatch"] == 0
    assert rep["tokens"] >= 2
    margin = float(np.expm1(2 * tol))
    for f in rep["flips"]:
        near = [x for x in (f.get("u_minus_alpha"), f.get("cdf_dist")) if x is not None]
        assert near and min(near) < margin, f
