"""Checks at full size: workload L (24 layers, dim 1024, vocabulary 16384, batch 128 with guidance = 256 physical
rows, window 32 -> 8192 token rows per forward, the launch configuration bench.py times) and the other full-size
configurations B (12 layers, no guidance), XL (36 layers, 24 x 24 tokens) and stress (L shape, batch 256, bimodal
prefix lengths).

The oracle needs seconds per image-round at these sizes, so element-wise parity is taken on sampled outputs: three
images per configuration (shortest, median, longest prefix) are followed in lockstep for four rounds, and one image
of L to completion, while the GPU runs the whole batch shape; everything else is checked through properties that
hold at any size.  The logit tolerance is not a formula: it is the oracle's own noise floor (the oracle against
its diagnostic form: fp32 instead of double sums, attention weights rounded to bf16), measured in the same test on
the first windows of the same images."""
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


def _check_against_floor(ctx, rep, model, w, toks, lab, k, ids, label):
    floor_max, floor_mean = G.floor_of(model, w, toks, lab, k, ids, norm_folded=ctx.fold_norm)
    G.check_logits_against_floor(rep, floor_max, floor_mean, label)
    assert rep["max_p_err"] <= 1e-6
    G.check_flips_explained(rep)


def test_fullsize_sampled_images_in_lockstep_with_the_oracle(big):
    """Three images -- shortest, median and longest prefix -- followed for four rounds while the GPU runs the whole
    batch shape: contexts of several pages, prefixes written by chunked pre-filling, cursors inside pages."""
    w, weights, ctx, toks, k, lab = big
    order = np.argsort(k, kind="stable")
    ids = sorted({int(order[0]), int(order[len(order) // 2]), int(order[-1])})
    model = O.Model(w.shape, weights)
    rep = G.lockstep(ctx, model, w, toks, k, lab, 23, image_ids=ids, max_rounds=4, park_others=False)
    assert rep["tokens"] >= 4 * len(ids)
    _check_against_floor(ctx, rep, model, w, toks, lab, k, ids, f"{w.name} ids {ids} k {[int(k[b]) for b in ids]}")


def test_fullsize_one_image_to_completion(big):
    """One image of workload L followed in lockstep until it is complete (40 tokens to generate), through the
    ragged last windows n < W, with the rest of the batch live beside it on the GPU."""
    w, weights, ctx, toks, k, lab = big
    if w.name != "L":
        pytest.skip("one configuration is enough for the run to completion")
    k2 = k.copy()
    b = 5
    k2[b] = w.shape.T - 40
    model = O.Model(w.shape, weights)
    rep = G.lockstep(ctx, model, w, toks, k2, lab, 29, image_ids=[b], park_others=False)
    assert rep["tokens"] == 40
    _check_against_floor(ctx, rep, model, w, toks, lab, k2, [b], f"{w.name} image {b} to completion")


def test_fullsize_greedy_verification_in_lockstep(big):
    """Greedy verification (Eq. 4) at full vocabulary and batch: two images of workload B followed for four rounds;
    an argmax that differs from the oracle's must be a near-tie of the oracle's own logits, which the per-flip
    replay establishes (the oracle's verification fed the GPU's probabilities reproduces the GPU's decision)."""
    w, weights, ctx, toks, k, lab = big
    if w.name != "B":
        pytest.skip("one configuration is enough for the greedy rule at full size")
    order = np.argsort(k, kind="stable")
    ids = sorted({int(order[0]), int(order[-1])})
    model = O.Model(w.shape, weights)
    rep = G.lockstep(ctx, model, w, toks, k, lab, 31, greedy=True, image_ids=ids, max_rounds=4, park_others=False)
    assert rep["tokens"] >= 4 * len(ids)
    _check_against_floor(ctx, rep, model, w, toks, lab, k, ids, f"{w.name} greedy ids {ids}")

